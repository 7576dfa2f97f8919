// ReduceScatter, AllGather, Broadcast and Reduce on the symmetric heap (paper Sec. V,
// "NCCL Collective Integration": the same low-latency primitives also give these
// collectives; Sec. III: AllReduce = ReduceScatter + AllGather = Reduce + Broadcast).
//
// All four are one-synchronisation pull kernels: slot c of every rank exchanges
// "input ready" signals with its peers (the same flag words and counters as the
// AllReduce kernels, so calls of any kind can alternate on one heap), then every
// rank reads what it needs from the peers' inputs and writes only its OWN output.
// Reductions are the rank-ordered binary32 sum with one narrowing, as everywhere.
#include "symar_device.cuh"
#include "symar_internal.h"

namespace symar {

enum : int { kOpReduceScatter = 0, kOpAllGather = 1, kOpBroadcast = 2, kOpReduce = 3 };

// ---- unit access: 16, 4 or 2 bytes, chosen by the common alignment of all offsets ----
template <int U> struct Unit;
template <> struct Unit<16> {
    uint4 v;
    __device__ static __forceinline__ Unit ld(const char *p) { Unit u; u.v = ld_peer(p); return u; }
};
template <> struct Unit<4> {
    uint32_t v;
    __device__ static __forceinline__ Unit ld(const char *p) { Unit u; u.v = ld_relaxed_u32(reinterpret_cast<const uint32_t *>(p)); return u; }
};
template <> struct Unit<2> {
    uint16_t v;
    __device__ static __forceinline__ Unit ld(const char *p)
    {
        Unit u;
        p = SYMAR_PTR(p, 2, kRegIn);
        asm volatile("ld.relaxed." SYMAR_SCOPE ".global.u16 %0, [%1];" : "=h"(u.v) : "l"(p) : "memory");
        return u;
    }
};

// store of the first `valid` bytes of a unit (valid is a multiple of 2, at most U)
__device__ __forceinline__ void st_unit(char *p, const Unit<16> &u, uint32_t valid)
{
    Words<4> w = {{u.v.x, u.v.y, u.v.z, u.v.w}};
    store_words<4>(p, w, valid);
}
__device__ __forceinline__ void st_unit(char *p, const Unit<4> &u, uint32_t valid)
{
    Words<1> w = {{u.v}};
    store_words<1>(p, w, valid);
}
__device__ __forceinline__ void st_unit(char *p, const Unit<2> &u, uint32_t)
{
    *SYMAR_PTR(reinterpret_cast<uint16_t *>(p), 2, kRegOut) = u.v;
}

template <typename E, int P>
__device__ __forceinline__ Unit<16> sum_units(const Unit<16> (&x)[P])
{
    uint4 v[P];
#pragma unroll
    for (int q = 0; q < P; ++q) v[q] = x[q].v;
    Unit<16> r;
    r.v = reduce_in_rank_order<E, P>(v);
    return r;
}
template <typename E, int P>
__device__ __forceinline__ Unit<4> sum_units(const Unit<4> (&x)[P])
{
    Words<1> w[P];
#pragma unroll
    for (int q = 0; q < P; ++q) w[q].w[0] = x[q].v;
    Unit<4> r;
    r.v = reduce_words_in_rank_order<E, P, 1>(w).w[0];
    return r;
}
template <typename E, int P>
__device__ __forceinline__ Unit<2> sum_units(const Unit<2> (&x)[P])     // one bf16 element
{
    float acc = __uint_as_float((uint32_t)x[0].v << 16);
#pragma unroll
    for (int q = 1; q < P; ++q) acc = __fadd_rn(acc, __uint_as_float((uint32_t)x[q].v << 16));
    __nv_bfloat16 h = __float2bfloat16_rn(acc);
    Unit<2> r;
    r.v = *reinterpret_cast<uint16_t *>(&h);
    return r;
}

struct CollArgs {
    KArgs    k;           // heap addressing, flags, limits (in_off / out_off / count unused fields aside)
    uint64_t bytes;       // bytes each rank reduces or copies per source (chunk, send size or message)
    int32_t  root;
};

template <typename E, int P, int OP, int U>
__device__ __forceinline__ void coll_body(const CollArgs &a, int r, uint64_t first, uint64_t step)
{
    const KArgs &k       = a.k;
    const uint64_t nunit = (a.bytes + U - 1) / U;
    char *out            = k.seg0 + (size_t)r * k.stride + k.out_off;
    for (uint64_t u = first; u < nunit; u += step) {
        const uint64_t off   = u * U;
        const uint32_t valid = a.bytes - off < (uint64_t)U ? (uint32_t)(a.bytes - off) : (uint32_t)U;
        if (OP == kOpReduceScatter || OP == kOpReduce) {
            const uint64_t src_off = k.in_off + (OP == kOpReduceScatter ? (uint64_t)r * a.bytes : 0) + off;
            Unit<U> x[P];
#pragma unroll
            for (int q = 0; q < P; ++q) x[q] = Unit<U>::ld(k.seg0 + (size_t)q * k.stride + src_off);
            st_unit(out + off, sum_units<E, P>(x), valid);
        } else if (OP == kOpAllGather) {
            Unit<U> x[P];
#pragma unroll
            for (int q = 0; q < P; ++q) x[q] = Unit<U>::ld(k.seg0 + (size_t)q * k.stride + k.in_off + off);
#pragma unroll
            for (int q = 0; q < P; ++q) st_unit(out + (uint64_t)q * a.bytes + off, x[q], valid);
        } else {
            st_unit(out + off, Unit<U>::ld(k.seg0 + (size_t)a.root * k.stride + k.in_off + off), valid);
        }
    }
}

template <typename E, int P, int OP>
__global__ void __launch_bounds__(kMaxThreads) coll_kernel(const CollArgs a)
{
    // input and output sizes per rank: ReduceScatter reads P chunks, AllGather writes P
    SYMAR_CHECK_BEGIN(a.k, P, OP == kOpReduceScatter ? a.bytes * P : a.bytes, OP == kOpAllGather ? a.bytes * P : a.bytes);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    const KArgs &k = a.k;
    const uint32_t *count = reinterpret_cast<const uint32_t *>(counters_near(k, r, c) + kCtrReady);
    if (k.pdl) {
        pdl_wait();
        pdl_launch_dependents();      // as in the one-shot AllReduce kernel: the successor may take its seats at once
    }

    uint32_t want;
    const bool ok = flag_exchange<P, false>(k, k.ready_off, kPairReady, count, r, c, false, true, want);
    __syncthreads();
    publish_u32(k, r, c, kCtrReady, want);
    if (!ok) return;
    if (OP == kOpReduce && r != a.root) return;          // only the root receives the sum

    const uint64_t first = (uint64_t)c * T + t, step = (uint64_t)C * T;
    if (k.variant == 16) coll_body<E, P, OP, 16>(a, r, first, step);
    else if (k.variant == 4) coll_body<E, P, OP, 4>(a, r, first, step);
    else if (E::kEpv == 8) coll_body<E, P, OP, 2>(a, r, first, step);     // bf16 element by element
}

using CollFn = void (*)(const CollArgs);

template <typename E, int P>
static CollFn pick_op(int op)
{
    switch (op) {
        case kOpReduceScatter: return coll_kernel<E, P, kOpReduceScatter>;
        case kOpAllGather:     return coll_kernel<E, P, kOpAllGather>;
        case kOpBroadcast:     return coll_kernel<E, P, kOpBroadcast>;
        case kOpReduce:        return coll_kernel<E, P, kOpReduce>;
    }
    return nullptr;
}
template <typename E>
static CollFn pick_coll(int op, int P)
{
    switch (P) {
        case 1: return pick_op<E, 1>(op);
        case 2: return pick_op<E, 2>(op);
        case 4: return pick_op<E, 4>(op);
        case 8: return pick_op<E, 8>(op);
    }
    return nullptr;
}

// Launch of one sibling collective.  `k` carries the heap addressing (as for the
// AllReduce kernels) with in_off / out_off set; unit = 16, 4 or 2 bytes.
static void coll_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute attr[2], int P, int ctas_per_rank, int threads,
                        bool pdl, bool cluster, cudaStream_t stream)
{
    cfg          = cudaLaunchConfig_t{};
    cfg.gridDim  = dim3((unsigned)ctas_per_rank, (unsigned)P, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.stream   = stream;
    cfg.attrs    = attr;
    cfg.numAttrs = 0;
    if (pdl) {
        attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
        ++cfg.numAttrs;
    }
    if (cluster && P > 1) {       // the ranks of a slot on SMs of one GPC (placement only, as for the AllReduce kernels)
        attr[cfg.numAttrs].id               = cudaLaunchAttributeClusterDimension;
        attr[cfg.numAttrs].val.clusterDim.x = 1;
        attr[cfg.numAttrs].val.clusterDim.y = (unsigned)P;
        attr[cfg.numAttrs].val.clusterDim.z = 1;
        ++cfg.numAttrs;
    }
}

cudaError_t launch_collective(int op, int dtype, int P, int ctas_per_rank, int threads, const KArgs &k,
                              uint64_t bytes, int root, int unit, cudaStream_t stream, bool cluster)
{
    CollFn fn = dtype == SYMAR_F32 ? pick_coll<F32>(op, P) : pick_coll<BF16>(op, P);
    if (!fn) return cudaErrorInvalidValue;
    CollArgs a;
    a.k         = k;
    a.k.variant = (uint32_t)unit;
    a.bytes     = bytes;
    a.root      = root;
    if (!k.pdl && !(cluster && P > 1)) {
        fn<<<dim3((unsigned)ctas_per_rank, (unsigned)P, 1), dim3((unsigned)threads, 1, 1), 0, stream>>>(a);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    coll_config(cfg, attr, P, ctas_per_rank, threads, k.pdl != 0, cluster, stream);
    return cudaLaunchKernelEx(&cfg, fn, a);
}

// clusters of one slot's P CTAs of a collective kernel that the device holds at once (0: none can be launched)
int collective_resident_clusters(int op, int dtype, int P, int threads)
{
    CollFn fn = dtype == SYMAR_F32 ? pick_coll<F32>(op, P) : pick_coll<BF16>(op, P);
    if (!fn || P < 2) return 0;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    coll_config(cfg, attr, P, 1, threads, false, true, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

// co-resident CTAs of a collective kernel at the given block size (they wait for one another)
int collective_resident(int op, int dtype, int P, int threads, int num_sms)
{
    CollFn fn = dtype == SYMAR_F32 ? pick_coll<F32>(op, P) : pick_coll<BF16>(op, P);
    int per_sm = 1;
    if (!fn || cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, 0) != cudaSuccess) per_sm = 1;
    return (per_sm > 0 ? per_sm : 1) * num_sms;
}

}  // namespace symar
