// allreduce_static(): the LL (data + flag) AllReduce for callers that must not
// allocate device memory.
//
// Who cannot allocate: code that runs where cudaMalloc is forbidden or unsafe --
// a callback in the middle of a latency-critical serving loop whose memory pool
// is frozen, a plugin loaded into a host process that gave it no allocator, code
// that may run while another thread captures a CUDA graph (an allocation then
// fails the capture), or an embedded deployment that sizes all device memory at
// start-up.  Such callers own their input and output buffers but have nowhere
// to put a symmetric heap with its LL scratch.
//
// Here the scratch lives in ONE file-scope __device__ array that every GPU
// which loads this library carries until the process exits (kStaticBytes, about
// 8 MiB).  Nothing is allocated or freed by this entry point, by the set-up it
// performs on first use, or by anything they call.
//
// What the array holds, and what persists between calls:
//   * per-slot iteration counters and the LL flags inside the scratch rows are
//     monotone sequence numbers.  They are MEANT to persist: a call's flag value
//     is one more than the last one used by the same CTA slot, so stale rows can
//     never look fresh, and nothing has to be cleared between calls.  (The array
//     starts zeroed when the module is loaded; 0 means "never written".)  Calls
//     with different rank counts advance different subsets of ranks, so each
//     rank count keeps its own set of counters, and the flag carries the rank
//     count in its top two bits: a row left by a P = 8 call can never satisfy
//     a P = 4 call.
//   * the caller's optional status word is the one thing that must start at
//     zero; the entry point clears it on the caller's stream before the launch.
// Every call on a device shares the array: calls that overlap on the GPU (two
// streams, or two host threads) race on it and must be serialised by the caller.
#include <cuda_runtime.h>

#include <atomic>

#include "symar_device.cuh"

namespace symar {
namespace {

// ---- limits ------------------------------------------------------------------------
constexpr uint32_t kStaticMaxVecs   = 2048;                 // 32 KiB per rank
constexpr uint32_t kStaticThreads   = 128;                  // fixed: slot c always owns vectors [128 c, 128 c + 128)
constexpr uint32_t kStaticSlots     = kStaticMaxVecs / kStaticThreads;
constexpr size_t   kStaticRowBytes  = (size_t)kStaticMaxVecs * 32;                       // one sender, one parity
constexpr size_t   kStaticRankBytes = (size_t)2 * kMaxRanks * kStaticRowBytes;           // 2 parities x P senders
constexpr size_t   kStaticCtrBytes  = 4096;                 // 4 rank counts x kMaxRanks x kStaticSlots x u64
constexpr size_t   kStaticBytes     = kStaticCtrBytes + (size_t)kMaxRanks * kStaticRankBytes;
static_assert(4 * kMaxRanks * kStaticSlots * sizeof(uint64_t) <= kStaticCtrBytes, "counters do not fit");

// log2 of the rank count: selects the counter set and tags the flag
template <int P> struct Log2;
template <> struct Log2<1> { static constexpr uint32_t v = 0; };
template <> struct Log2<2> { static constexpr uint32_t v = 1; };
template <> struct Log2<4> { static constexpr uint32_t v = 2; };
template <> struct Log2<8> { static constexpr uint32_t v = 3; };

// 32-bit flag of iteration n for rank count 2^lg: never 0, top two bits = lg
__device__ __forceinline__ uint32_t static_flag(uint64_t n, uint32_t lg)
{
    return (lg << 30) | (1u + (uint32_t)(n % 0x3fffffffull));
}

// The scratch.  In HOST code this name is only a handle for cudaGetSymbolAddress;
// it is not a device address and must never be handed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

struct StaticArgs {
    const char    *in;          // rank q's input at in + q * pitch
    char          *out;         // rank r's output at out + r * pitch
    uint64_t       pitch;
    uint64_t       nvec;
    unsigned char *scratch;     // device address of g_static_scratch
    uint32_t      *status;      // caller's status word or nullptr
    uint64_t       spin_ns;
    uint32_t       tail_bytes;
};

// One-iteration LL AllReduce (paper Sec. IV "LL", Sec. V example kernel); same
// arithmetic and flag protocol as the heap-based LL kernel, other addressing.
template <typename E, int P>
__global__ void __launch_bounds__(kStaticThreads) ll_static_kernel(const StaticArgs a)
{
#ifdef SYMAR_CHECK
    if (threadIdx.x == 0) {       // checking build: the caller's rows and the two parts of the static array
        CheckCtx &cc = check_ctx();
        const uint64_t bytes = a.tail_bytes ? (a.nvec - 1) * 16 + a.tail_bytes : a.nvec * 16;
        cc.base = nullptr;
        cc.nreg = 0;
        cc.nranks = 0;
        cc.stride = 1;
        cc.ctl    = nullptr;
        cc.status = a.status;
        cc.nabs   = 4;
        cc.alo[0] = a.in;   cc.ahi[0] = a.in + (uint64_t)(P - 1) * a.pitch + bytes;  cc.akind[0] = kRegIn;
        cc.alo[1] = a.out;  cc.ahi[1] = a.out + (uint64_t)(P - 1) * a.pitch + bytes; cc.akind[1] = kRegOut;
        cc.alo[2] = reinterpret_cast<const char *>(a.scratch);
        cc.ahi[2] = cc.alo[2] + kStaticCtrBytes;                                     cc.akind[2] = kRegCtr;
        cc.alo[3] = cc.ahi[2];  cc.ahi[3] = cc.alo[2] + kStaticBytes;                cc.akind[3] = kRegLL;
    }
    __syncthreads();
#endif
    const int c = blockIdx.x, r = blockIdx.y;
    const uint32_t t = threadIdx.x;
    constexpr uint32_t lg = Log2<P>::v;
    uint64_t *ep = SYMAR_PTR(reinterpret_cast<uint64_t *>(a.scratch) + ((size_t)lg * kMaxRanks + r) * kStaticSlots + c, 8,
                             kRegCtr);
    const uint64_t n = ld_relaxed_u64(ep) + 1;
    const uint32_t e = static_flag(n, lg);
    const uint64_t v = (uint64_t)c * kStaticThreads + t;
    unsigned char *rows = a.scratch + kStaticCtrBytes;
    // receiver q, parity, sender s, half h, vector v
    auto row = [&](int q, int s) {
        return rows + (size_t)q * kStaticRankBytes + ((size_t)(n & 1) * kMaxRanks + s) * kStaticRowBytes;
    };
    bool failed = false;
    if (v < a.nvec) {
        uint4 x;
        if (a.tail_bytes != 0 && v == a.nvec - 1) {
            // The caller's buffer may end with the message: read only the valid
            // bytes of a partial last vector (the rest is sent as zeros and never stored).
            const uint16_t *src =
                SYMAR_PTR(reinterpret_cast<const uint16_t *>(a.in + (size_t)r * a.pitch + v * 16), a.tail_bytes, kRegIn);
            uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int b = 0; b < 8; ++b)
                if ((uint32_t)b < a.tail_bytes / 2) w[b >> 1] |= (uint32_t)src[b] << ((b & 1) * 16);
            x = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
            x = ld_own(a.in + (size_t)r * a.pitch + v * 16);
        }
        const uint64_t hi_e = (uint64_t)e << 32;
        const uint64_t d0 = hi_e | x.x, d1 = hi_e | x.y, d2 = hi_e | x.z, d3 = hi_e | x.w;
#pragma unroll
        for (int q = 0; q < P; ++q) {
            if (q == r) continue;
            unsigned char *dst = row(q, r) + v * 16;
            st_relaxed_v2u64(dst, d0, d1);
            st_relaxed_v2u64(dst + (size_t)kStaticMaxVecs * 16, d2, d3);
        }
        uint4 xs[P];
        unsigned need = ((1u << P) - 1u) & ~(1u << r);
        Spin spin;
        while (need != 0) {
            U64x2 lo[P], hi[P];
#pragma unroll
            for (int q = 0; q < P; ++q) {
                if (need >> q & 1u) {
                    const unsigned char *src = row(r, q) + v * 16;
                    lo[q] = ld_relaxed_v2u64(src);
                    hi[q] = ld_relaxed_v2u64(src + (size_t)kStaticMaxVecs * 16);
                }
            }
#pragma unroll
            for (int q = 0; q < P; ++q) {
                if (need >> q & 1u) {
                    const bool here = (uint32_t)(lo[q].a >> 32) == e && (uint32_t)(lo[q].b >> 32) == e &&
                                      (uint32_t)(hi[q].a >> 32) == e && (uint32_t)(hi[q].b >> 32) == e;
                    if (here) {
                        xs[q] = make_uint4((uint32_t)lo[q].a, (uint32_t)lo[q].b, (uint32_t)hi[q].a, (uint32_t)hi[q].b);
                        need &= ~(1u << q);
                    }
                }
            }
            if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                failed = true;
                break;
            }
        }
        if (!failed) {
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q == r) xs[q] = x;
            store_result(a.out + (size_t)r * a.pitch, v, reduce_in_rank_order<E, P>(xs), a.nvec, a.tail_bytes);
        } else if (a.status) {
            atomicCAS(a.status, 0u, (uint32_t)SYMAR_ERR_TIMEOUT);
        }
    }
    __syncthreads();          // every thread has read the counter before it moves
    if (t == 0) *ep = n;
}

using StaticFn = void (*)(const StaticArgs);

template <typename E>
StaticFn pick_static(int P)
{
    switch (P) {
        case 1: return ll_static_kernel<E, 1>;
        case 2: return ll_static_kernel<E, 2>;
        case 4: return ll_static_kernel<E, 4>;
        case 8: return ll_static_kernel<E, 8>;
    }
    return nullptr;
}

// Device address of the scratch, looked up once per device.  cudaGetSymbolAddress
// answers for the CURRENT device, so the cache is indexed by it.  Two host threads
// may make their first call on a device at the same time: both look the address up,
// both store the same value, and the atomic makes either store safe to read.
constexpr int kMaxDevices = 64;
std::atomic<unsigned char *> g_scratch_addr[kMaxDevices];

// All CTAs of a call wait for one another, so the largest launch (kStaticSlots CTAs for
// each of kMaxRanks ranks) must fit on the device at once; checked with the address.
int scratch_for_current_device(unsigned char **addr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SYMAR_ERR_CUDA;
    unsigned char *known = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (known == nullptr) {
        int sms = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ll_static_kernel<BF16, kMaxRanks>, (int)kStaticThreads,
                                                          0) != cudaSuccess) {
            cudaGetLastError();
            return SYMAR_ERR_CUDA;
        }
        if ((long)sms * per_sm < (long)kStaticSlots * kMaxRanks) return SYMAR_ERR_UNSUPPORTED;
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return SYMAR_ERR_CUDA;
        }
        known = static_cast<unsigned char *>(p);
        g_scratch_addr[dev].store(known, std::memory_order_release);
    }
    *addr = known;
    return SYMAR_OK;
}

}  // namespace
}  // namespace symar

extern "C" int allreduce_static(const void *in, void *out, size_t rank_pitch_bytes, int P, size_t count,
                                symar_dtype_t dtype, unsigned int *device_status, void *cuda_stream)
{
    using namespace symar;
    if (!in || !out) return SYMAR_ERR_INVAL;
    if (P != 1 && P != 2 && P != 4 && P != 8) return SYMAR_ERR_INVAL;
    if (dtype != SYMAR_F32 && dtype != SYMAR_BF16) return SYMAR_ERR_INVAL;
    const size_t es = dtype == SYMAR_F32 ? 4 : 2;
    if (count > SYMAR_STATIC_MAX_BYTES / es) return SYMAR_ERR_UNSUPPORTED;     // beyond the fixed scratch
    const size_t bytes = count * es;
    if (((uintptr_t)in | (uintptr_t)out | rank_pitch_bytes) & 15) return SYMAR_ERR_INVAL;
    if (P > 1 && rank_pitch_bytes < (bytes + 15) / 16 * 16) return SYMAR_ERR_INVAL;
    {
        // out-of-place: the P input rows and the P output rows must not overlap
        const uintptr_t i0 = (uintptr_t)in, i1 = i0 + (size_t)(P - 1) * rank_pitch_bytes + bytes;
        const uintptr_t o0 = (uintptr_t)out, o1 = o0 + (size_t)(P - 1) * rank_pitch_bytes + bytes;
        if (bytes != 0 && i0 < o1 && o0 < i1) return SYMAR_ERR_INVAL;
    }
    if (count == 0) return SYMAR_OK;

    unsigned char *scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);       // first call on a device: symbol look-up
    if (rc != SYMAR_OK) return rc;

    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (device_status && cudaMemsetAsync(device_status, 0, sizeof(unsigned int), s) != cudaSuccess) {
        cudaGetLastError();
        return SYMAR_ERR_CUDA;
    }
    StaticArgs a;
    a.in         = static_cast<const char *>(in);
    a.out        = static_cast<char *>(out);
    a.pitch      = rank_pitch_bytes;
    a.nvec       = (bytes + 15) / 16;
    a.scratch    = scratch;
    a.status     = device_status;
    a.spin_ns    = 200000000ull;       // 0.2 s: far beyond any call, short enough not to hold a shared GPU
    a.tail_bytes = (uint32_t)(bytes % 16);
    StaticFn fn  = dtype == SYMAR_F32 ? pick_static<F32>(P) : pick_static<BF16>(P);
    const unsigned ctas = (unsigned)((a.nvec + kStaticThreads - 1) / kStaticThreads);
    fn<<<dim3(ctas, (unsigned)P, 1), dim3(kStaticThreads, 1, 1), 0, s>>>(a);
    if (cudaGetLastError() != cudaSuccess) return SYMAR_ERR_CUDA;
    return SYMAR_OK;
}
