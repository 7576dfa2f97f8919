// Host side of libsymar: the symmetric heap, argument checking, the per-size
// selector with its autotuner, and the C ABI declared in include/symar.h.
// Every step of the collective itself runs in the kernels of symar_kernels.cu;
// there is no host or library fallback.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <tuple>
#include <chrono>
#include <vector>

#include "symar_internal.h"

namespace symar {

struct LaunchCfg {
    int ctas    = 0;   // per rank; 0 = not set
    int threads = 0;
    int variant = -1;  // kernel variant bits; -1 = not set
};

constexpr int kBuckets = 40;   // bucket b holds messages of (2^(b-1), 2^b] bytes per rank
constexpr int kAlgos   = 8;    // indexed by symar_algo_t
constexpr int kLastAlgo = SYMAR_TWOSHOT_ATOMIC;
constexpr int kLastTuned = SYMAR_TWOSHOT_SENTINEL;   // the tuner and AUTO stay with the bit-reproducible algorithms
static bool is_push(int algo) { return algo >= SYMAR_LL && algo <= SYMAR_TWOSHOT_SENTINEL; }   // per-slot scratch and epochs
static KernelFn any_kernel_for(int algo, int dtype, int P, bool dbg)
{
    return algo == SYMAR_TWOSHOT_ATOMIC ? atomic_kernel_for(dtype, P, dbg) : kernel_for(algo, dtype, P, dbg);
}
static bool is_twoshot_push(int algo) { return algo == SYMAR_TWOSHOT_LL || algo == SYMAR_TWOSHOT_SENTINEL; }

struct Tuned {
    bool      valid = false;
    int       best_algo[kBuckets];
    LaunchCfg cfg[kAlgos][kBuckets];
    double    us[kAlgos][kBuckets];
    int       lo_bucket = 0, hi_bucket = -1;
    bool      have[kBuckets] = {};     // buckets tuned one at a time (allreduce_autotune_size)
};

static thread_local std::string g_last_cuda_error;

// which half of the chip every SM of a device sits on: measured once per device and process
constexpr int kMaxDevices = 64;
struct DevicePlace { bool tried = false, ok = false; uint64_t sm_half[4] = {0, 0, 0, 0}; };
static DevicePlace g_place[kMaxDevices];
static std::mutex  g_place_mutex;

static int cuda_fail(cudaError_t e, const char *what)
{
    g_last_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    return SYMAR_ERR_CUDA;
}
#define CU(call)                                          \
    do {                                                  \
        cudaError_t e_ = (call);                          \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

}  // namespace symar

using namespace symar;

struct symheap {
    int       P              = 0;
    size_t    bytes_per_rank = 0;
    Layout    L{};
    char     *mem   = nullptr;   // heap base (control block)
    bool      owns  = false;
    char     *seg0  = nullptr;
    uint32_t *ctl   = nullptr;
    int       device  = 0;
    int       num_sms = 0;
    int       max_smem = 48 * 1024;   // opt-in dynamic shared memory per CTA
    uint64_t  spin_ns = 200000000ull;    // 200 ms: hundreds of times the longest call (a 256 MiB message takes 0.65 ms)
    bool      pdl          = true;    // programmatic dependent launch of every kernel
    int       env_algo     = 0;       // SYMAR_ALGO override of SYMAR_AUTO, 0 = none
    bool      cluster_on   = true;    // SYMAR_CLUSTER=0: never launch a slot's ranks as a thread-block cluster
    bool      debug_log    = false;   // SYMAR_DEBUG=1: one stderr line per call
    long      tune_timed[kAlgos] = {};   // tuner: graphs timed per algorithm, and the seconds that took
    double    tune_secs[kAlgos]  = {};
    bool      tune_exhaustive = false;   // SYMAR_TUNE=exhaustive: the tuner prunes nothing
    int       tune_rotate = 0;        // tuner: > 0 = every call of a timing graph has its own buffers (that many pairs)
    bool      placed   = false;       // sm_half / home were measured cleanly
    bool      place_on = true;        // readers take the copy of their own L2 half (SYMAR_PLACE=0 / symar_set_placement)
    uint64_t  sm_half[4] = {0, 0, 0, 0};
    uint64_t  home = 0;
    size_t    scratch_limit = 0;      // push algorithms: payload bytes per rank and iteration, 0 = all there is
    int       dbg_mute     = -1;
    unsigned  dbg_seed     = 0;
    unsigned  dbg_delay_ns = 0;
    bool      dbg_span     = false;
    LaunchCfg forced[kAlgos];
    unsigned  variant[kAlgos] = {};
    bool      variant_forced[kAlgos] = {};
    Tuned     tuned[2];
    int       last_algo = 0, last_ctas = 0, last_threads = 0;
    unsigned  last_variant = 0;
    size_t    last_smem = 0;
    std::map<std::tuple<const void *, int>, int> resident;   // (kernel, threads) -> CTAs co-resident
    // allreduce_host() on large messages: copy streams and events of the chunk pipeline (made on first use)
    cudaStream_t h2d = nullptr, d2h = nullptr;
    std::vector<cudaEvent_t> pipe_ev;
};

namespace symar {

static size_t elem_size(int dtype) { return dtype == SYMAR_F32 ? 4 : 2; }
static bool   valid_P(int P) { return P == 1 || P == 2 || P == 4 || P == 8; }
static bool   dbg_on(const symheap *h) { return h->dbg_mute >= 0 || h->dbg_delay_ns != 0 || h->dbg_span; }

static int bucket_of(size_t bytes)
{
    int b = 0;
    while (b < kBuckets - 1 && ((size_t)1 << b) < bytes) ++b;
    return b;
}

// CTAs of the given kernel and block size that fit on the device at once.  The
// CTAs of different ranks wait for one another, so a grid larger than this
// could leave a waiting CTA holding the SM that the CTA it waits for needs.
static int max_resident(symheap *h, KernelFn fn, int threads, size_t smem = 0)
{
    auto key = std::make_tuple((const void *)fn, threads + (int)(smem << 4));
    auto it  = h->resident.find(key);
    if (it != h->resident.end()) return it->second;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, smem) != cudaSuccess) per_sm = 1;
    int n = std::max(1, per_sm) * h->num_sms;
    h->resident[key] = n;
    return n;
}

// Clusters of one slot's P CTAs that fit on the device at once (0: such a cluster cannot be launched).
static int max_clusters(symheap *h, KernelFn fn, int threads, size_t smem)
{
    auto key = std::make_tuple((const void *)fn, -(threads + (int)(smem << 4)) - 1);
    auto it  = h->resident.find(key);
    if (it != h->resident.end()) return it->second;
    const int n = max_resident_clusters(fn, h->P, threads, smem);
    if (h->debug_log)
        std::fprintf(stderr, "symar: clusters of %d CTAs x %d threads resident at once: %d%s\n", h->P, threads, n,
                     n < 0 ? " (minus the CUDA error of the occupancy query)" : "");
    h->resident[key] = n;
    return n;
}

static int round_threads(uint64_t want)
{
    int t = 32;
    while (t < (int)kMaxThreads && (uint64_t)t < want) t *= 2;
    return t;
}

// Variant bits of the bulk two-shot kernel: pipeline depth and tile size.
static int bulk_variant(int stages, int tile_log2_over_4k) { return (stages << 8) | (tile_log2_over_4k << 12); }

// LL, single-iteration kernel: the largest message it covers (64 slots x 256 threads x 8 bytes), and
// the default hold-back of the first poll in steps of 64 cycles.  A poll that leaves before the row has
// landed costs a whole further round trip, one that leaves late costs its lateness; the best hold-back is
// the store-to-visibility time less what the kernel does anyway between its stores and its first poll.
// Measured with each slot's ranks launched as a cluster (sweeps at P = 8, 4, 2 from 128 B to 128 KiB; the
// minimum is sharp: 0.06 to 0.15 us lost one step of 128 cycles beside it): nothing up to 256 B and
// between two ranks up to 4 KiB, 128 cycles up to 16 KiB, then growing with the rows in flight to a full
// hop (768 cycles).
constexpr uint64_t kLLSmallMaxBytes = (uint64_t)kLLSlots * kLLMaxThreads * 8;
static unsigned ll_default_gap(int P, uint64_t bytes)
{
    if (bytes <= 256) return 0;
    if (P >= 8) return bytes <= (16u << 10) ? 2 : (bytes <= (32u << 10) ? 12 : 8);
    if (P == 4) return bytes <= (16u << 10) ? 2 : (bytes <= (32u << 10) ? 4 : (bytes <= (64u << 10) ? 6 : 8));
    return bytes <= 4096 ? 0 : 2;
}

// Whether the P CTAs of a slot are launched as one thread-block cluster (on SMs of one GPC, hence on one
// half of the chip) when nobody said otherwise.  Measured on B200, A/B on one heap (64-call graphs): the
// data+flag protocol gains 0.2 to 0.5 us at nearly every size and rank count (its rows are written and
// polled across the chip otherwise); one-shot and two-shot gain 0.03 to 0.13 us while the CTAs are few
// and lose as much or far more once they fill the chip (a cluster must find P free SMs in one GPC).
static bool cluster_default(int algo, int P, uint64_t bytes)
{
    if (P < 2 || bytes >= kBulkMinVec * 16) return false;
    if (is_push(algo)) return true;                      // sentinel and the push two-shots gain 0.2 to 1 us
    if (algo == SYMAR_ONESHOT)
        return P == 8 ? bytes <= (128u << 10) : (P == 4 ? bytes > (16u << 10) && bytes <= (2u << 20) : bytes >= (128u << 10));
    if (algo == SYMAR_TWOSHOT)
        return P == 8 ? bytes <= (128u << 10) : (P == 4 ? bytes <= (256u << 10) : bytes >= (16u << 10));
    return false;
}

// Launch shape when neither the caller nor the tuner fixed one.  Every rule here restates what the
// tuner chose on B200 for 2, 4 and 8 ranks from 128 B to 256 MiB; an untuned call stays within a few
// percent of the tuned one (measured: at most 7 %, typically 0 to 3 %).
static LaunchCfg default_shape(symheap *h, int algo, uint64_t nvec, KernelFn fn)
{
    LaunchCfg c;
    c.variant = 0;
    const int P = h->P;
    const uint64_t bytes = nvec * 16;
    const uint64_t work  = (algo == SYMAR_TWOSHOT || is_twoshot_push(algo)) ? (nvec + P - 1) / P
                                                                            : nvec;   // vectors per rank partition
    if (algo == SYMAR_TWOSHOT && nvec >= kBulkMinVec) {
        // Bandwidth regime: the register kernel with 512 threads per SM in all, in as many CTAs per rank as
        // half or a quarter of the SMs (all ranks' CTAs together are then a whole number per SM, an even
        // load; 64 CTAs per rank among eight leave some SMs with three and some with four): 37 x 256 among
        // eight ranks, 74 x 256 among four,
        // 74 x 512 between two.  The bulk-copy kernel comes within 3 % with about 100 CTAs in total, each
        // with one 64 KiB stage ahead of the one it reduces, and the tuner still times it; from 4 to 16 MiB,
        // where repeated calls find their buffers in L2, it is 10 to 40 % behind.
        c.variant = 4;
        c.threads = P >= 4 ? 256 : 512;
        c.ctas    = std::max(1, std::min(h->num_sms * 512 / P / c.threads, (int)kMaxCtas));
        return c;
    }
    if (algo == SYMAR_TWOSHOT) {
        // Latency regime of two-shot: one unit per thread; at most 128 / P CTAs per rank, blocks growing to
        // 512 threads before threads take a second unit; 8192 threads per rank at most (16384 between two).
        // Among eight ranks a unit is 8 bytes up to 512 KiB (measured 0.15 to 0.45 us ahead of 16 bytes from
        // 16 KiB on; no gain among four or two ranks, none from 1 MiB).
        uint64_t units = work;
        const uint64_t budget = P == 2 ? 16384 : 8192;
        if (nvec >= kCyclicMinVec) {
            // from 1 MiB blocks of 8 KiB are dealt to the ranks and a thread moves 32 bytes per trip: half as
            // many CTAs per rank as SMs (an even load, see above), small ones.  Measured among eight ranks at
            // 1 MiB: 74 CTAs of 64 threads 4.7 us, 64 of 64 5.2 us, 16 of 512 6.5 us; at 2 MiB: 16 to 18 CTAs of
            // 512 threads 7.1 us, 37 of 256 7.4 to 8.4 us, 74 of 128 7.9 us.
            const uint64_t n    = std::min((work + 1) / 2, budget);
            const uint64_t half = (uint64_t)std::max(1, std::min(h->num_sms / 2, (int)kMaxCtas));
            if (n <= half * 64) {
                c.threads = 64;
                c.ctas    = (int)half;
            } else if (P == 8) {
                c.threads = 512;
                c.ctas    = (int)std::max<uint64_t>(1, half / 4);
            } else {
                c.threads = 128;
                c.ctas    = (int)half;
            }
            return c;
        }
        if (P == 8 && bytes <= (512u << 10)) {
            c.variant = 0x40;
            units     = work * 2;
        }
        const uint64_t cap_c  = (uint64_t)std::max(1, 128 / P);
        uint64_t T = units <= 128 ? (uint64_t)round_threads(std::max<uint64_t>(units, 64)) : 128;
        while (T < kMaxThreads && (units + T - 1) / T > cap_c) T *= 2;
        uint64_t C = std::min((units + T - 1) / T, cap_c);
        if (C * T > budget) T = std::max<uint64_t>(128, budget / C);
        c.threads = (int)T;
        c.ctas    = (int)std::max<uint64_t>(1, C);
        return c;
    }
    if (algo == SYMAR_ONESHOT) {
        // Small messages are bound by the per-thread instruction chain, so a thread takes 8 bytes up to
        // 64 KiB (4 up to 256 B, where that still fills a warp) and 16 above.  One unit per thread: one CTA
        // up to 256 units, blocks of 128 up to half as many CTAs per rank as SMs, then larger blocks as far as
        // the kernel's registers let all ranks' CTAs be resident together; beyond that equal passes.
        const int narrow = bytes <= 256 ? 2 : (bytes <= (64u << 10) ? 1 : 0);
        c.variant = narrow << 8;
        const uint64_t units = work << narrow;
        if (units <= 256) {
            c.threads = round_threads(units);
            c.ctas    = 1;
            return c;
        }
        uint64_t best_cover = 0;
        const uint64_t half = (uint64_t)std::max(1, std::min(h->num_sms / 2, (int)kMaxCtas));
        for (int T : {128, 256, 512}) {
            const uint64_t res = fn ? (uint64_t)std::max(1, max_resident(h, fn, T, 0) / P) : half;
            const uint64_t C   = std::min<uint64_t>({(units + T - 1) / T, half, res});
            const uint64_t cover = std::min(units, C * T);
            if (cover > best_cover) {
                best_cover = cover;
                c.threads  = T;
                c.ctas     = (int)C;
            }
        }
        const uint64_t per_pass = (uint64_t)c.ctas * c.threads;
        const uint64_t passes   = (units + per_pass - 1) / per_pass;
        c.ctas = (int)std::max<uint64_t>(1, (units + passes * c.threads - 1) / (passes * c.threads));
        return c;
    }
    uint64_t units = work;
    if (algo == SYMAR_LL && bytes <= kLLSmallMaxBytes) {
        // the single-iteration kernel with 8 bytes of payload per thread (measured ahead of 16 bytes
        // per thread at every size it covers), first poll held back by the default for this traffic
        c.variant = 0x100 | (ll_default_gap(P, bytes) << 12);
        units     = work * 2;
        c.threads = units <= 64 ? round_threads(units) : (units < 2048 ? 64 : (units <= 8192 ? 128 : 256));
        c.ctas    = (int)std::min<uint64_t>((units + c.threads - 1) / c.threads, (uint64_t)kLLSlots);
        return c;
    }
    c.threads = units >= 2048 ? 128 : round_threads(std::max<uint64_t>(units / 16, 32));
    uint64_t ctas = (units + c.threads - 1) / c.threads;
    const uint64_t cap = is_push(algo) ? (uint64_t)kLLSlots : (uint64_t)std::max(1, 2 * h->num_sms / P);
    c.ctas = (int)std::max<uint64_t>(1, std::min(ctas, cap));
    return c;
}

static LaunchCfg default_cfg(symheap *h, int algo, uint64_t nvec, KernelFn fn)
{
    LaunchCfg c = default_shape(h, algo, nvec, fn);
    if (cluster_default(algo, h->P, nvec * 16)) c.variant |= (int)kVarCluster;
    return c;
}

// Before autotuning.  Measured on B200: with ranks that share one L2 the pull
// one-shot wins from about 1 KiB up to 256 KiB per rank, two-shot above; LL saves
// one dependent round trip and pays for it with P - 1 flagged stores and polls per
// thread, which is a gain only while those are few.
static int default_algo(int P, size_t bytes)
{
    // the data+flag protocol leads at the smallest sizes (Sec. VII Obs. 1); measured here, with flag
    // and counter reads placed on the reader's L2 half, each slot's ranks launched as a cluster and the
    // first poll held back as above: between two ranks 1.18 to 1.43 us from 128 B to 128 KiB against
    // one-shot's 1.37 to 1.62; among four 1.18 to 1.50 us up to 32 KiB against 1.46 to 1.53; among eight
    // 1.40 against 1.43 us at 128 B, level at 4 KiB, behind elsewhere
    if (P == 2 && bytes <= kLLSmallMaxBytes) return SYMAR_LL;
    if (P == 4 && bytes <= (32u << 10)) return SYMAR_LL;
    if (P == 8 && bytes <= 256) return SYMAR_LL;
    // one-shot reads P times the bytes two-shot does and saves its second synchronisation: the
    // break-even moves up fourfold each time the rank count halves (measured 256 KiB, 1 MiB, 4 to 8 MiB)
    const size_t limit = (size_t)(256u << 10) * (size_t)(64 / (P * P));
    if (bytes <= limit) return SYMAR_ONESHOT;
    return SYMAR_TWOSHOT;
}

struct Plan {
    int       algo;
    LaunchCfg cfg;
    KernelFn  fn;
    size_t    smem = 0;     // dynamic shared memory of the launch
    bool      cluster = false;   // the ranks of a slot as one thread-block cluster
    KArgs     args;
};

// Resolves algorithm and launch shape and fills the kernel arguments.
static int make_plan(symheap *h, size_t in_off, size_t out_off, size_t count, int dtype, int algo, Plan *p)
{
    const size_t es    = elem_size(dtype);
    const size_t bytes = count * es;
    const uint64_t nvec = (bytes + 15) / 16;
    const Tuned &tn    = h->tuned[dtype];
    // the size's own bucket if it was tuned, else the nearest bucket of a full table
    int b = bucket_of(bytes);
    bool tuned = tn.have[b];
    if (!tuned && tn.valid) {
        b     = std::min(std::max(b, tn.lo_bucket), tn.hi_bucket);
        tuned = true;
    }

    if (algo == SYMAR_AUTO) algo = h->env_algo ? h->env_algo : (tuned ? tn.best_algo[b] : default_algo(h->P, bytes));

    LaunchCfg cfg = default_cfg(h, algo, nvec, algo == SYMAR_ONESHOT ? any_kernel_for(algo, dtype, h->P, dbg_on(h)) : nullptr);
    if (tuned && tn.cfg[algo][b].ctas > 0) cfg = tn.cfg[algo][b];
    if (h->forced[algo].ctas > 0) cfg.ctas = h->forced[algo].ctas;
    if (h->forced[algo].threads > 0) cfg.threads = h->forced[algo].threads;
    if (h->variant_forced[algo]) cfg.variant = (int)h->variant[algo];
    if (cfg.variant < 0) cfg.variant = 0;
    bool cluster       = ((unsigned)cfg.variant & kVarCluster) != 0 && h->P > 1 && h->cluster_on;
    const unsigned var = (unsigned)cfg.variant & ~kVarCluster;      // what the kernel sees

    cfg.threads = std::min<int>(std::max(32, (cfg.threads + 31) / 32 * 32),
                                is_twoshot_push(algo) ? (int)kPushTwoshotMaxThreads
                                                      : (algo == SYMAR_LL ? (int)kLLMaxThreads : (int)kMaxThreads));
    KArgs &a = p->args;
    std::memset(&a, 0, sizeof a);
    KernelFn fn = any_kernel_for(algo, dtype, h->P, dbg_on(h));
    p->smem     = 0;
    if (algo == SYMAR_TWOSHOT_ATOMIC) {
        // one 8-thread group per 128-byte line of 31 elements; a chunk must fit in one scratch half
        const uint64_t ch = (count + h->P - 1) / h->P;
        const uint64_t nl = (ch + kAtLinePayload - 1) / kAtLinePayload;
        if (nl > at_lines_per_half(h->P)) return SYMAR_ERR_UNSUPPORTED;
        if (h->forced[algo].threads <= 0 && !(tuned && tn.cfg[algo][b].ctas > 0))
            cfg.threads = nl * 8 >= 8192 ? 512 : (nl * 8 >= 256 ? 256 : round_threads(std::max<uint64_t>(nl * 8, 32)));
        cfg.threads = std::max(32, (cfg.threads + 31) / 32 * 32);
        if (h->forced[algo].ctas <= 0 && !(tuned && tn.cfg[algo][b].ctas > 0))
            cfg.ctas = (int)std::max<uint64_t>(
                1, std::min<uint64_t>((nl * 8 + cfg.threads - 1) / cfg.threads, (uint64_t)std::max(1, h->num_sms / h->P)));
    }
    // bandwidth regime of two-shot: the bulk-copy kernel (the test hooks live in
    // the register kernel only)
    if (algo == SYMAR_TWOSHOT && nvec >= kBulkMinVec && !dbg_on(h) && !(var & 4u)) {
        fn          = bulk_kernel_for(dtype, h->P);
        const unsigned v = var;
        a.tile_vecs = 256u << ((v >> 12) & 3u);                       // 4, 8, 16 or 32 KiB tiles
        a.stages    = ((v >> 8) & 7u) ? ((v >> 8) & 7u) : 2u;
        while (a.stages > 2 && bulk_smem_bytes(h->P, a.tile_vecs, a.stages) > (size_t)h->max_smem) --a.stages;
        while (a.tile_vecs > 256 && bulk_smem_bytes(h->P, a.tile_vecs, a.stages) > (size_t)h->max_smem)
            a.tile_vecs /= 2;
        p->smem     = bulk_smem_bytes(h->P, a.tile_vecs, a.stages);
    }
    if (!fn) return SYMAR_ERR_INVAL;
    const int cap_slots = (is_push(algo) || algo == SYMAR_TWOSHOT_ATOMIC) ? kLLSlots : kMaxCtas;
    // LL: a message that the launch covers with one unit per thread takes the straight-line
    // single-iteration kernel (variant bit 9 keeps the general one)
    if (algo == SYMAR_LL && !(var & 0x200u) && !h->scratch_limit) {
        const int words      = (var & 0x100u) ? 2 : 4;
        const uint64_t units = (bytes + 4 * words - 1) / (4 * words);
        const uint64_t need  = (units + cfg.threads - 1) / cfg.threads;
        KernelFn sfn = ll_small_kernel_for(dtype, h->P, words, dbg_on(h));
        if (sfn && need <= (uint64_t)cfg.ctas && need <= (uint64_t)cap_slots &&
            need <= (uint64_t)std::max(1, max_resident(h, sfn, cfg.threads, 0) / h->P)) {
            fn       = sfn;
            cfg.ctas = (int)need;
        }
    }
    const int cap_res = std::max(1, max_resident(h, fn, cfg.threads, p->smem) / h->P);
    cfg.ctas = std::max(1, std::min({cfg.ctas, cap_slots, cap_res}));
    // all clusters must be resident together, like all CTAs; where they are not, the plain launch of the
    // same shape (the bulk-copy kernel is never launched in clusters)
    if (cluster && (p->smem != 0 || max_clusters(h, fn, cfg.threads, p->smem) < cfg.ctas)) cluster = false;
    cfg.variant = (int)(var | (cluster ? kVarCluster : 0u));
    p->cluster  = cluster;

    a.seg0       = h->seg0;
    a.stride     = h->L.stride;
    a.in_off     = in_off;
    a.out_off    = out_off;
    a.count      = count;
    a.nvec       = nvec;
    a.ll_off     = h->L.ll_off;
    a.sn_off     = h->L.sn_off;
    a.at_off     = h->L.at_off;
    a.ready_off  = h->L.ready_off;
    a.done_off   = h->L.done_off;
    a.epoch_off  = h->L.epoch_off;
    a.ctl        = h->ctl;
    a.spin_ns    = h->spin_ns;
    a.tail_bytes = (uint32_t)(bytes % 16);
    a.variant    = var;
    a.pdl        = h->pdl ? 1u : 0u;
    a.dbg_mute   = h->dbg_mute;
    a.dbg_seed   = h->dbg_seed;
    a.dbg_delay_ns = h->dbg_delay_ns;
    a.dbg_span   = h->dbg_span ? 1u : 0u;
    if (h->placed && h->place_on) {
        std::memcpy(a.sm_half, h->sm_half, sizeof a.sm_half);
        a.home = h->home;
    }
    if (algo == SYMAR_TWOSHOT) {
        const bool cyclic = nvec >= kCyclicMinVec && !(var & 1u);
        a.blk_log2 = cyclic ? kCyclicLog2 : kOneChunk;
        a.wide     = cyclic && ((in_off | out_off) % 32 == 0) && !(var & 2u);
    }
    if (is_push(algo)) {
        // every CTA takes `cv` positions per iteration; iterations alternate sub-buffers.  The
        // two-shot forms walk chunk positions and keep half of a scratch row for each phase.
        const uint64_t span    = is_twoshot_push(algo) ? (nvec + h->P - 1) / h->P : nvec;
        const uint64_t max_cv  = is_twoshot_push(algo) ? kLLSlotVecs / 2 : kLLSlotVecs;
        const uint64_t per_cta = (span + cfg.ctas - 1) / cfg.ctas;
        a.cv    = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(per_cta, max_cv));
        if (h->scratch_limit) {      // a smaller scratch buffer: fewer positions per iteration, more iterations
            const uint64_t per_iter = std::max<uint64_t>(1, h->scratch_limit / 16 / (is_twoshot_push(algo) ? h->P : 1));
            a.cv = (uint32_t)std::max<uint64_t>(1, std::min<uint64_t>(a.cv, per_iter / cfg.ctas));
        }
        a.iters = (uint32_t)((span + (uint64_t)a.cv * cfg.ctas - 1) / ((uint64_t)a.cv * cfg.ctas));
    }
    p->algo = algo;
    p->cfg  = cfg;
    p->fn   = fn;
    return SYMAR_OK;
}

static int check_buffers(const symheap *h, const void *in, const void *out, size_t count, int dtype,
                         size_t *in_off, size_t *out_off)
{
    if (!h || !in || !out) return SYMAR_ERR_INVAL;
    if (dtype != SYMAR_F32 && dtype != SYMAR_BF16) return SYMAR_ERR_INVAL;
    const char *pi = (const char *)in, *po = (const char *)out;
    if (pi < h->seg0 || po < h->seg0) return SYMAR_ERR_INVAL;
    const size_t io = pi - h->seg0, oo = po - h->seg0;
    const size_t bytes = count * elem_size(dtype);
    if (count != 0 && bytes / count != elem_size(dtype)) return SYMAR_ERR_INVAL;   // overflow
    if ((io | oo) & 15) return SYMAR_ERR_INVAL;
    if (io > h->bytes_per_rank || bytes > h->bytes_per_rank - io) return SYMAR_ERR_INVAL;
    if (oo > h->bytes_per_rank || bytes > h->bytes_per_rank - oo) return SYMAR_ERR_INVAL;
    if (bytes != 0 && io < oo + bytes && oo < io + bytes) return SYMAR_ERR_INVAL;    // out-of-place only
    *in_off  = io;
    *out_off = oo;
    return SYMAR_OK;
}

static int run(symheap *h, const void *in, void *out, size_t count, int dtype, int algo, cudaStream_t s)
{
    size_t io = 0, oo = 0;
    int rc = check_buffers(h, in, out, count, dtype, &io, &oo);
    if (rc != SYMAR_OK) return rc;
    if (algo < SYMAR_AUTO || algo > kLastAlgo) return SYMAR_ERR_INVAL;
    if (count == 0) return SYMAR_OK;
    Plan p;
    rc = make_plan(h, io, oo, count, dtype, algo, &p);
    if (rc != SYMAR_OK) return rc;
    cudaError_t e = launch_kernel(p.fn, h->P, p.cfg.ctas, p.cfg.threads, p.smem, p.args, s, p.cluster);
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    h->last_algo    = p.algo;
    h->last_ctas    = p.cfg.ctas;
    h->last_threads = p.cfg.threads;
    h->last_variant = (unsigned)p.cfg.variant;      // with the cluster bit, which no kernel sees
    h->last_smem    = p.smem;
    if (h->debug_log)
        std::fprintf(stderr, "symar: allreduce count=%zu dtype=%d algo=%d grid=(%d,%d) block=%d variant=%#x smem=%zu pdl=%d\n",
                     count, dtype, p.algo, p.cfg.ctas, h->P, p.cfg.threads, (unsigned)p.cfg.variant, p.smem, (int)h->pdl);
    return SYMAR_OK;
}

// ---- sibling collectives --------------------------------------------------------------
// op: 0 ReduceScatter (in: P*n per rank, out: n), 1 AllGather (in: n, out: P*n),
//     2 Broadcast, 3 Reduce (in: n, out: n).  n = `count` elements.
static int run_collective(symheap *h, int op, const void *in, void *out, size_t count, int dtype, int root,
                          cudaStream_t s)
{
    if (!h || !in || !out) return SYMAR_ERR_INVAL;
    if (dtype != SYMAR_F32 && dtype != SYMAR_BF16) return SYMAR_ERR_INVAL;
    if ((op == 2 || op == 3) && (root < 0 || root >= h->P)) return SYMAR_ERR_INVAL;
    const size_t es = elem_size(dtype);
    if (count != 0 && (count * es) / count != es) return SYMAR_ERR_INVAL;
    const size_t bytes = count * es;
    if (bytes > h->bytes_per_rank) return SYMAR_ERR_INVAL;
    const size_t in_total  = op == 0 ? bytes * h->P : bytes;
    const size_t out_total = op == 1 ? bytes * h->P : bytes;
    const char *pi = (const char *)in, *po = (const char *)out;
    if (pi < h->seg0 || po < h->seg0) return SYMAR_ERR_INVAL;
    const size_t io = pi - h->seg0, oo = po - h->seg0;
    if ((io | oo) & 15) return SYMAR_ERR_INVAL;
    if (io > h->bytes_per_rank || in_total > h->bytes_per_rank - io) return SYMAR_ERR_INVAL;
    if (oo > h->bytes_per_rank || out_total > h->bytes_per_rank - oo) return SYMAR_ERR_INVAL;
    if (bytes != 0 && io < oo + out_total && oo < io + in_total) return SYMAR_ERR_INVAL;     // out-of-place only
    if (count == 0) return SYMAR_OK;

    // widest unit that every per-rank offset is aligned to
    const bool strided = op == 0 || op == 1;              // chunk q starts at q * bytes
    const int unit = (!strided || bytes % 16 == 0) ? 16 : (bytes % 4 == 0 ? 4 : 2);
    const uint64_t units = (bytes + unit - 1) / unit;
    int threads = units >= 2048 ? 128 : round_threads(std::max<uint64_t>(units / 16, 32));
    const int cap = std::max(1, std::min({(int)kMaxCtas, collective_resident(op, dtype, h->P, threads, h->num_sms) / h->P,
                                          std::max(1, 2 * h->num_sms / h->P)}));
    const int ctas = (int)std::max<uint64_t>(1, std::min<uint64_t>((units + threads - 1) / threads, (uint64_t)cap));

    KArgs a;
    std::memset(&a, 0, sizeof a);
    a.seg0      = h->seg0;
    a.stride    = h->L.stride;
    a.in_off    = io;
    a.out_off   = oo;
    a.count     = count;
    a.ready_off = h->L.ready_off;
    a.done_off  = h->L.done_off;
    a.epoch_off = h->L.epoch_off;
    a.ctl       = h->ctl;
    a.spin_ns   = h->spin_ns;
    a.pdl       = h->pdl ? 1u : 0u;
    a.dbg_mute  = -1;
    if (h->placed && h->place_on) {
        std::memcpy(a.sm_half, h->sm_half, sizeof a.sm_half);
        a.home = h->home;
    }
    // each slot's ranks as one cluster while the CTAs are few (the one-shot AllReduce's rule: these kernels
    // have its structure; measured -0.03 to -0.13 us up to 64 KiB among eight ranks), if all clusters can be
    // resident together
    bool cluster = h->cluster_on && cluster_default(SYMAR_ONESHOT, h->P, op == 0 ? in_total : out_total);
    if (cluster) {
        auto key = std::make_tuple((const void *)(intptr_t)(0x1000 + op * 16 + dtype), -threads - 1);
        auto it  = h->resident.find(key);
        const int n = it != h->resident.end() ? it->second
                                              : (h->resident[key] = collective_resident_clusters(op, dtype, h->P, threads));
        cluster = n >= ctas;
    }
    cudaError_t e = launch_collective(op, dtype, h->P, ctas, threads, a, bytes, root, unit, s, cluster);
    if (e != cudaSuccess) return cuda_fail(e, "collective launch");
    h->last_algo    = SYMAR_ONESHOT;
    h->last_ctas    = ctas;
    h->last_threads = threads;
    h->last_variant = (unsigned)unit;
    h->last_smem    = 0;
    return SYMAR_OK;
}

// ---- autotuner ---------------------------------------------------------------------

// Median per-call time (us) of K back-to-back calls captured in one graph.
// `give_up_us` > 0: a candidate whose first three replays all take longer than that is not worth
// the remaining replays (its fastest replay is returned).
static int time_calls(symheap *h, cudaStream_t s, size_t count, int dtype, int algo, int K, int reps,
                      double *us_out, double give_up_us = 0.0)
{
    const size_t bytes = count * elem_size(dtype);
    const auto wall0   = std::chrono::steady_clock::now();
    struct Tally {
        symheap *h; int algo; std::chrono::steady_clock::time_point t0;
        ~Tally() { ++h->tune_timed[algo]; h->tune_secs[algo] += std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count(); }
    } tally{h, algo, wall0};
    // Warm: every call on the same input and output.  Streaming (tune_rotate pairs): call k reads and writes its
    // own pair of buffers, as the calls of a decode step do; the graph then holds one call per pair.
    const size_t slice = round_up(bytes, kAlign);
    const int pairs    = h->tune_rotate > 0 ? h->tune_rotate : 1;
    if (h->tune_rotate > 0) K = pairs;
    cudaGraph_t graph;
    cudaGraphExec_t exec;
    CU(cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal));
    int rc = SYMAR_OK;
    for (int k = 0; k < K && rc == SYMAR_OK; ++k)
        rc = run(h, h->seg0 + (size_t)(k % pairs) * slice, h->seg0 + (size_t)(pairs + k % pairs) * slice, count, dtype, algo, s);
    cudaError_t ce = cudaStreamEndCapture(s, &graph);
    if (rc != SYMAR_OK) {
        if (ce == cudaSuccess) cudaGraphDestroy(graph);
        return rc;
    }
    if (ce != cudaSuccess) return cuda_fail(ce, "cudaStreamEndCapture");
    ce = cudaGraphInstantiate(&exec, graph, 0);
    if (ce != cudaSuccess) {
        cudaGraphDestroy(graph);
        return cuda_fail(ce, "cudaGraphInstantiate");
    }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    std::vector<float> ms(reps);
    cudaGraphLaunch(exec, s);   // warm
    for (int i = 0; i < reps; ++i) {
        cudaEventRecord(e0, s);
        cudaGraphLaunch(exec, s);
        cudaEventRecord(e1, s);
        cudaEventSynchronize(e1);
        cudaEventElapsedTime(&ms[i], e0, e1);
        if (i == 2 && give_up_us > 0.0 && (double)std::min({ms[0], ms[1], ms[2]}) * 1000.0 / K > give_up_us) {
            ms.assign(reps, std::min({ms[0], ms[1], ms[2]}));
            break;
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaGraphExecDestroy(exec);
    cudaGraphDestroy(graph);
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return cuda_fail(ce, "autotune timing");
    std::sort(ms.begin(), ms.end());
    *us_out = (double)ms[reps / 2] * 1000.0 / K;
    return SYMAR_OK;
}

// Times algorithms, launch shapes and kernel variants on messages of `bytes` per rank and records
// the winners in bucket b of `tn`.
//
// With `prev` >= 0 (the bucket tuned just before, one size step down) the search is pruned by
// what that bucket showed, unless the heap asks for the exhaustive search:
//   * an algorithm that moves more bytes per rank than the winner does (the push forms: 2 to 4 times
//     the payload through scratch; above 1 MiB also one-shot: P times the reads) and that lost by
//     more than 1.5 x one step down is not timed again -- its traffic grows as fast as the winner's
//     or faster, so it cannot come back (Table I's volume column); its row reads "not timed";
//   * above 4 MiB the launch shapes of an algorithm are searched around its winner one step down
//     (CTA counts from half to four times, every block size), since a message twice as large
//     wants about as many CTAs or the next larger count;
//   * a shape whose first three replays are all a quarter slower than the algorithm's best so far
//     is not replayed further.
static int tune_bucket(symheap *h, int dtype, int b, size_t bytes, cudaStream_t s, Tuned &tn, int prev = -1)
{
    static const int kThreads[] = {64, 128, 256, 512};
    static const int kCtas[]    = {1, 2, 4, 8, 10, 12, 15, 16, 18, 24, 32, 37, 48, 64, 74};
    const size_t es     = elem_size(dtype);
    const size_t count  = bytes / es;
    const uint64_t nvec = (bytes + 15) / 16;
    const int K    = bytes <= (1u << 20) ? 24 : (bytes <= (16u << 20) ? 6 : 2);
    const int reps = 7;
    const bool prune = prev >= 0 && !h->tune_exhaustive;
    LaunchCfg saved[kAlgos];
    unsigned saved_variant[kAlgos];
    bool saved_forced[kAlgos];
    for (int a = 0; a < kAlgos; ++a) {
        saved[a]         = h->forced[a];
        saved_variant[a] = h->variant[a];
        saved_forced[a]  = h->variant_forced[a];
    }
    int rc = SYMAR_OK;
    double best_us = 1e30;
    tn.best_algo[b] = SYMAR_ONESHOT;
    double prev_best = 1e30;
    if (prune)
        for (int a = SYMAR_ONESHOT; a <= kLastTuned; ++a) prev_best = std::min(prev_best, tn.us[a][prev]);
    for (int algo = SYMAR_ONESHOT; algo <= kLastTuned && rc == SYMAR_OK; ++algo) {
        tn.us[algo][b]  = 1e30;
        tn.cfg[algo][b] = LaunchCfg{};
        if (is_push(algo) && bytes > (4u << 20)) continue;   // scratch traffic through L2: hopeless there
        if (algo != SYMAR_TWOSHOT && bytes > (32u << 20)) continue;   // only two-shot moves the minimum of bytes
        if (prune && bytes > (64u << 10) && (is_push(algo) || (algo == SYMAR_ONESHOT && bytes > (1u << 20))) &&
            tn.us[algo][prev] > 1.5 * prev_best)
            continue;                                        // lost one step down, and its traffic grows at least as fast
        const uint64_t work = (algo == SYMAR_TWOSHOT || is_twoshot_push(algo)) ? (nvec + h->P - 1) / h->P : nvec;
        // kernel variants worth timing: the default; for two-shot in the bandwidth
        // regime the bulk kernel's tile sizes and depths, and the register kernel
        std::vector<int> variants = {0};
        const bool bulk = algo == SYMAR_TWOSHOT && nvec >= kBulkMinVec;
        if (bulk)
            variants = {bulk_variant(2, 1), bulk_variant(3, 1), bulk_variant(2, 2), bulk_variant(3, 0),
                        bulk_variant(4, 0), 4};
        else if (algo == SYMAR_ONESHOT && bytes <= (1u << 20)) {
            // 16, 8 or 4 bytes per thread, each where it has ever won (exhaustive searches chose 4 bytes up to
            // 256 B only, 8 bytes up to 64 KiB, 16 bytes from 2 KiB)
            variants.clear();
            if (bytes >= 2048 || h->tune_exhaustive) variants.push_back(0);
            if (bytes <= (256u << 10) || h->tune_exhaustive) variants.push_back(0x100);
            if (bytes <= 4096 || h->tune_exhaustive) variants.push_back(0x200);
        }
        else if (algo == SYMAR_TWOSHOT && nvec < kCyclicMinVec)
            variants = {0, 0x40};                    // 16 or 8 bytes per thread and trip
        else if (algo == SYMAR_LL && bytes <= kLLSmallMaxBytes) {
            // 8 bytes of payload per thread with the first poll held back by the default for this
            // size, by 128 cycles less and more, by half a hop more, and not at all; 16 bytes per thread
            const int g = (int)ll_default_gap(h->P, bytes);
            variants = {0x100 | (g << 12)};
            for (int alt : {g - 2, g + 2, g + 6, 0})
                if (alt >= 0 && alt <= 15 && alt != g &&
                    std::find(variants.begin(), variants.end(), 0x100 | (alt << 12)) == variants.end())
                    variants.push_back(0x100 | (alt << 12));
            if (bytes >= 4096) variants.push_back(g << 12);
        } else if (algo == SYMAR_LL && bytes <= (256u << 10))
            variants = {0, 0x100};                   // general kernel: 16 or 8 bytes of payload per thread
        struct Cand { double us; LaunchCfg cfg; };
        std::vector<Cand> cands;                     // the first pass's shapes, for a second look
        // the neighbourhood of this algorithm's winner one step down
        // (above 4 MiB only, where every call is long and one kernel form covers all sizes: below, calls
        // are short, and the best shape still moves with the unit width and, at 1 MiB, with the change
        // from contiguous chunks to blocks dealt round-robin -- measured 5 to 8 % lost at 1 to 4 MiB)
        const LaunchCfg near =
            (prune && bytes > (4u << 20) && tn.cfg[algo][prev].ctas > 0) ? tn.cfg[algo][prev] : LaunchCfg{};
        if (!bulk && cluster_default(algo, h->P, bytes))
            for (int &v : variants) v |= (int)kVarCluster;     // launched as the built-in rule would; the second look tries the other way
        for (int var : variants) {
            // threads a shape needs: one per unit of this variant
            const uint64_t units = bulk ? work : (work << ((var >> 8) & 3)) << ((algo == SYMAR_TWOSHOT && (var & 0x40)) ? 1 : 0);
            for (int T : kThreads) {
                if (bulk && var != 4 && T != 128 && T != 256) continue;
                for (int C : kCtas) {
                    // skip shapes with far more threads than vectors, except the smallest
                    if ((uint64_t)C * T > 2 * units && !(C == 1 && T == 64)) continue;
                    // and shapes that would leave each thread hundreds of units
                    if (!bulk && units / ((uint64_t)C * T) > 4096) continue;
                    if (bulk && (C * h->P < 48)) continue;
                    if (near.ctas > 0 && (2 * C < near.ctas || C > 4 * near.ctas)) continue;
                    h->forced[algo]         = LaunchCfg{C, T, var};
                    h->variant[algo]        = (unsigned)var;
                    h->variant_forced[algo] = true;
                    Plan p;
                    if (make_plan(h, 0, round_up(bytes, kAlign), count, dtype, algo, &p) != SYMAR_OK) continue;
                    if (p.cfg.ctas != C || p.cfg.threads != T) continue;   // clamped: a duplicate of another shape
                    double us = 0;
                    // a shape a quarter slower than this algorithm's best so far is dropped after three replays
                    rc = time_calls(h, s, count, dtype, algo, K, reps, &us,
                                    h->tune_exhaustive || tn.us[algo][b] > 1e29 ? 0.0 : 1.25 * tn.us[algo][b]);
                    if (rc != SYMAR_OK) break;
                    cands.push_back(Cand{us, LaunchCfg{C, T, var}});
                    // a larger launch must win by more than the timing noise (1.5 %) to displace a smaller one
                    const LaunchCfg &cur = tn.cfg[algo][b];
                    const bool larger    = cur.ctas > 0 && (long)C * T > (long)cur.ctas * cur.threads;
                    if (us < tn.us[algo][b] * (larger ? 0.985 : 1.0)) {
                        tn.us[algo][b]  = us;
                        tn.cfg[algo][b] = LaunchCfg{C, T, var};
                    }
                }
                if (rc != SYMAR_OK) break;
            }
            if (rc != SYMAR_OK) break;
        }
        // Bandwidth regime: the best shapes lie within a percent or two of one another, less than the
        // noise of the short first pass.  Time the four fastest again, longer, and keep the winner.
        if (bulk && rc == SYMAR_OK && cands.size() > 1) {
            std::sort(cands.begin(), cands.end(), [](const Cand &x, const Cand &y) { return x.us < y.us; });
            cands.resize(std::min<size_t>(cands.size(), 4));
            double best = 1e30;
            for (const Cand &cd : cands) {
                h->forced[algo]         = cd.cfg;
                h->variant[algo]        = (unsigned)cd.cfg.variant;
                h->variant_forced[algo] = true;
                double us = 0;
                rc = time_calls(h, s, count, dtype, algo, 4, 15, &us);
                if (rc != SYMAR_OK) break;
                if (us < best) {
                    best            = us;
                    tn.us[algo][b]  = us;
                    tn.cfg[algo][b] = cd.cfg;
                }
            }
        }
        // Latency regime: shapes of an algorithm that could win this size differ by a timer step or two
        // (0.03 us per call in a 24-call graph).  Time its three fastest again in a graph twice as long
        // and keep the winner, so that the choice does not hang on one noisy replay.
        if (!bulk && rc == SYMAR_OK && cands.size() > 1 && tn.us[algo][b] <= 1.2 * best_us) {
            std::sort(cands.begin(), cands.end(), [](const Cand &x, const Cand &y) { return x.us < y.us; });
            cands.resize(std::min<size_t>(cands.size(), 3));
            // ... the two fastest also with the slot's ranks launched the other way (as one cluster, or not)
            if (h->P > 1)
                for (size_t i = 0, n = std::min<size_t>(cands.size(), 2); i < n; ++i) {
                    Cand other = cands[i];
                    other.cfg.variant ^= (int)kVarCluster;
                    cands.push_back(other);
                }
            double best = 1e30;
            for (const Cand &cd : cands) {
                h->forced[algo]         = cd.cfg;
                h->variant[algo]        = (unsigned)cd.cfg.variant;
                h->variant_forced[algo] = true;
                double us = 0;
                rc = time_calls(h, s, count, dtype, algo, 2 * K, 9, &us);
                if (rc != SYMAR_OK) break;
                if (us < best) {
                    best            = us;
                    tn.us[algo][b]  = us;
                    tn.cfg[algo][b] = cd.cfg;
                }
            }
        }
        h->forced[algo]         = saved[algo];
        h->variant[algo]        = saved_variant[algo];
        h->variant_forced[algo] = saved_forced[algo];
        if (tn.us[algo][b] < best_us) {
            best_us         = tn.us[algo][b];
            tn.best_algo[b] = algo;
        }
    }
    for (int a = 0; a < kAlgos; ++a) {
        h->forced[a]         = saved[a];
        h->variant[a]        = saved_variant[a];
        h->variant_forced[a] = saved_forced[a];
    }
    return rc;
}

// only_bytes == 0: the whole power-of-two grid; else just the bucket of that size, at that size
static int autotune(symheap *h, int dtype, size_t only_bytes, int rotate = 0)
{
    const size_t es = elem_size(dtype);
    // input and output side by side; with `rotate` pairs of buffers, that many of each
    const size_t fit = h->bytes_per_rank / 2 / (size_t)(rotate > 0 ? rotate : 1) / kAlign * kAlign;
    if (fit < 16) return SYMAR_ERR_INVAL;
    cudaStream_t s;
    CU(cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking));
    const Tuned saved_tuned = h->tuned[dtype];
    int rc = SYMAR_OK;
    if (only_bytes) {
        const size_t bytes = only_bytes / es * es;
        if (bytes < es || bytes > fit) {
            cudaStreamDestroy(s);
            return SYMAR_ERR_INVAL;
        }
        Tuned tn      = saved_tuned;
        const int b   = bucket_of(bytes);
        tn.have[b]    = false;
        h->tuned[dtype].valid = false;                 // time with defaults, not with a stale table
        std::memset(h->tuned[dtype].have, 0, sizeof h->tuned[dtype].have);
        h->tune_rotate = rotate;
        rc = tune_bucket(h, dtype, b, bytes, s, tn);
        h->tune_rotate = 0;
        tn.have[b] = rc == SYMAR_OK;
        cudaStreamSynchronize(s);
        cudaStreamDestroy(s);
        h->tuned[dtype] = rc == SYMAR_OK ? tn : saved_tuned;
        return rc;
    }
    Tuned tn;
    const size_t max_bytes = std::min<size_t>(fit, (size_t)64 << 20);
    tn.lo_bucket = 4;
    tn.hi_bucket = 4;
    while (tn.hi_bucket + 1 < kBuckets && ((size_t)1 << (tn.hi_bucket + 1)) <= max_bytes) ++tn.hi_bucket;
    h->tuned[dtype].valid = false;
    std::memset(h->tuned[dtype].have, 0, sizeof h->tuned[dtype].have);
    for (int b = tn.lo_bucket; b <= tn.hi_bucket && rc == SYMAR_OK; ++b)
        rc = tune_bucket(h, dtype, b, (size_t)1 << b, s, tn, b > tn.lo_bucket ? b - 1 : -1);
    cudaStreamSynchronize(s);
    cudaStreamDestroy(s);
    if (h->debug_log)
        for (int a = SYMAR_ONESHOT; a < kAlgos; ++a)
            if (h->tune_timed[a])
                std::fprintf(stderr, "symar: tuner, algorithm %d: %ld graphs timed in %.2f s\n", a, h->tune_timed[a], h->tune_secs[a]);
    if (rc != SYMAR_OK) {
        h->tuned[dtype] = saved_tuned;
        return rc;
    }
    tn.valid = true;
    for (int b = 0; b < kBuckets; ++b) tn.have[b] = saved_tuned.have[b] && (b < tn.lo_bucket || b > tn.hi_bucket);
    // keep individually tuned buckets outside the grid
    for (int b = 0; b < kBuckets; ++b)
        if (tn.have[b]) {
            tn.best_algo[b] = saved_tuned.best_algo[b];
            for (int a = 0; a < kAlgos; ++a) {
                tn.cfg[a][b] = saved_tuned.cfg[a][b];
                tn.us[a][b]  = saved_tuned.us[a][b];
            }
        }
    h->tuned[dtype] = tn;
    return SYMAR_OK;
}

static int create_common(symheap_t **heap, int P, size_t bytes_per_rank, void *mem, size_t mem_bytes, bool owns)
{
    Layout L = make_layout(P, bytes_per_rank);
    if (mem_bytes < L.total) return SYMAR_ERR_NOMEM;
    if (((uintptr_t)mem & (kAlign - 1)) != 0) return SYMAR_ERR_INVAL;
    symheap *h = new (std::nothrow) symheap;
    if (!h) return SYMAR_ERR_NOMEM;
    h->P = P;
    h->bytes_per_rank = bytes_per_rank;
    h->L    = L;
    h->mem  = (char *)mem;
    h->owns = owns;
    h->seg0 = h->mem + kCtlBytes;
    h->ctl  = (uint32_t *)h->mem;
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device);
    // Where the SMs and this heap's flag and counter lines sit on the chip's two L2 halves (measured once
    // per device and once per heap, in the heap's own scratch, before everything is zeroed).
    if (const char *v = std::getenv("SYMAR_PLACE")) h->place_on = std::atoi(v) != 0;
    if (e == cudaSuccess && h->place_on && h->device >= 0 && h->device < kMaxDevices) {
        unsigned char *scratch = reinterpret_cast<unsigned char *>(h->seg0 + L.ll_off);
        bool ok = false;
        {
            std::lock_guard<std::mutex> lock(g_place_mutex);
            DevicePlace &dp = g_place[h->device];
            if (!dp.tried) {
                e = place_measure_sms(scratch, h->num_sms, h->max_smem, dp.sm_half, &dp.ok);
                dp.tried = e == cudaSuccess;
            }
            ok = dp.ok;
            std::memcpy(h->sm_half, dp.sm_half, sizeof h->sm_half);
        }
        if (e == cudaSuccess && ok) e = place_measure_heap(h->seg0, L.stride, P, L, h->sm_half, scratch, &h->home, &h->placed);
    }
    if (e == cudaSuccess) e = cudaMemset(h->mem, 0, kCtlBytes);
    for (int q = 0; q < P && e == cudaSuccess; ++q) {
        e = cudaMemset(h->seg0 + (size_t)q * L.stride + L.ll_off, 0, L.seg_bytes - L.ll_off);
        if (e == cudaSuccess) e = cudaMemset(h->seg0 + (size_t)q * L.stride + L.sn_off, 0xff, L.sn_bytes);
    }
    // Load every kernel this heap can launch now, so that a first call made
    // during stream capture does not trigger lazy module loading there.
    // The bulk kernel's dynamic shared memory is what the opt-in limit leaves beside its
    // static shared memory (none in the regular build).
    int bulk_static = 0;
    for (int dt = SYMAR_F32; dt <= SYMAR_BF16 && e == cudaSuccess; ++dt) {
        cudaFuncAttributes attr;
        e = cudaFuncGetAttributes(&attr, bulk_kernel_for(dt, P));
        if (e == cudaSuccess) bulk_static = std::max(bulk_static, (int)attr.sharedSizeBytes);
    }
    h->max_smem -= bulk_static;
    for (int algo = SYMAR_ONESHOT; algo <= kLastAlgo && e == cudaSuccess; ++algo)
        for (int dt = SYMAR_F32; dt <= SYMAR_BF16 && e == cudaSuccess; ++dt) {
            cudaFuncAttributes attr;
            e = cudaFuncGetAttributes(&attr, any_kernel_for(algo, dt, P, false));
            if (e == cudaSuccess && algo == SYMAR_TWOSHOT)
                // opt in to the large dynamic shared memory now (not during a capture)
                e = cudaFuncSetAttribute(bulk_kernel_for(dt, P), cudaFuncAttributeMaxDynamicSharedMemorySize, h->max_smem);
            if (e == cudaSuccess && algo == SYMAR_LL)
                for (int words = 2; words <= 4 && e == cudaSuccess; words += 2)
                    e = cudaFuncGetAttributes(&attr, ll_small_kernel_for(dt, P, words, false));
        }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        delete h;
        return cuda_fail(e, "heap initialisation");
    }
    // Environment overrides (read once per heap): SYMAR_SPIN_LIMIT_US bounds every
    // device-side wait; SYMAR_ALGO = oneshot | twoshot | ll | ... replaces SYMAR_AUTO's choice;
    // SYMAR_PDL = 0 turns programmatic dependent launch off; SYMAR_CTAS_PER_RANK and
    // SYMAR_THREADS fix the launch shape of every algorithm; SYMAR_DEBUG = 1 logs every
    // call's resolved algorithm and shape to stderr; SYMAR_TUNE = exhaustive makes
    // allreduce_autotune time every algorithm and shape at every size (no pruning);
    // SYMAR_PLACE = 0 (read above) skips the placement measurement: every reader takes copy 0.
    if (const char *v = std::getenv("SYMAR_SPIN_LIMIT_US")) {
        const long us = std::atol(v);
        if (us > 0) h->spin_ns = (uint64_t)us * 1000ull;
    }
    if (const char *v = std::getenv("SYMAR_ALGO")) {
        const std::string a(v);
        h->env_algo = a == "oneshot" ? SYMAR_ONESHOT : a == "twoshot" ? SYMAR_TWOSHOT : a == "ll" ? SYMAR_LL : a == "sentinel" ? SYMAR_SENTINEL
                      : a == "twoshot_ll" ? SYMAR_TWOSHOT_LL : a == "twoshot_sentinel" ? SYMAR_TWOSHOT_SENTINEL
                      : a == "twoshot_atomic" ? SYMAR_TWOSHOT_ATOMIC : 0;
    }
    if (const char *v = std::getenv("SYMAR_PDL")) h->pdl = std::atoi(v) != 0;
    if (const char *v = std::getenv("SYMAR_CTAS_PER_RANK")) {
        const int c = std::atoi(v);
        if (c > 0 && c <= kMaxCtas)
            for (int a = SYMAR_ONESHOT; a <= kLastAlgo; ++a) h->forced[a].ctas = c;
    }
    if (const char *v = std::getenv("SYMAR_THREADS")) {
        const int t = std::atoi(v);
        if (t > 0 && t <= (int)kMaxThreads)
            for (int a = SYMAR_ONESHOT; a <= kLastAlgo; ++a) h->forced[a].threads = t;
    }
    if (const char *v = std::getenv("SYMAR_DEBUG")) h->debug_log = std::atoi(v) != 0;
    if (const char *v = std::getenv("SYMAR_CLUSTER")) h->cluster_on = std::atoi(v) != 0;
    if (const char *v = std::getenv("SYMAR_TUNE")) h->tune_exhaustive = std::string(v) == "exhaustive";
    *heap = h;
    return SYMAR_OK;
}

}  // namespace symar

// ---- C ABI ---------------------------------------------------------------------------

extern "C" {

size_t symheap_required_bytes(int P, size_t bytes_per_rank)
{
    if (!valid_P(P)) return 0;
    return make_layout(P, bytes_per_rank).total;
}

int symheap_create(symheap_t **heap, int P, size_t bytes_per_rank)
{
    if (!heap || !valid_P(P) || bytes_per_rank == 0) return SYMAR_ERR_INVAL;
    const size_t total = make_layout(P, bytes_per_rank).total;
    void *mem = nullptr;
    cudaError_t e = cudaMalloc(&mem, total);
    if (e == cudaErrorMemoryAllocation) {
        cudaGetLastError();
        return SYMAR_ERR_NOMEM;
    }
    if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc");
    int rc = create_common(heap, P, bytes_per_rank, mem, total, true);
    if (rc != SYMAR_OK) cudaFree(mem);
    return rc;
}

int symheap_create_on(symheap_t **heap, int P, size_t bytes_per_rank, void *device_mem, size_t device_bytes)
{
    if (!heap || !valid_P(P) || bytes_per_rank == 0 || !device_mem) return SYMAR_ERR_INVAL;
    return create_common(heap, P, bytes_per_rank, device_mem, device_bytes, false);
}

int symheap_destroy(symheap_t *heap)
{
    if (!heap) return SYMAR_ERR_INVAL;
    int rc = SYMAR_OK;
    if (heap->owns) {
        cudaError_t e = cudaFree(heap->mem);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaFree");
    }
    for (cudaEvent_t ev : heap->pipe_ev) cudaEventDestroy(ev);
    if (heap->h2d) cudaStreamDestroy(heap->h2d);
    if (heap->d2h) cudaStreamDestroy(heap->d2h);
    delete heap;
    return rc;
}

int symheap_info(const symheap_t *heap, symheap_info_t *info)
{
    if (!heap || !info) return SYMAR_ERR_INVAL;
    info->P                = heap->P;
    info->bytes_per_rank   = heap->bytes_per_rank;
    info->user_bytes       = heap->L.user_bytes;
    info->ll_scratch_bytes = heap->L.ll_bytes;
    info->sentinel_scratch_bytes = heap->L.sn_bytes;
    info->atomic_scratch_bytes = heap->L.at_bytes;
    info->flag_bytes       = heap->L.seg_bytes - heap->L.ready_off;
    info->stride           = heap->L.stride;
    info->total_bytes      = heap->L.total;
    info->base             = heap->seg0;
    return SYMAR_OK;
}

void *symheap_rank_ptr(const symheap_t *heap, int rank, size_t offset)
{
    if (!heap || rank < 0 || rank >= heap->P || offset >= heap->L.user_bytes) return nullptr;
    return heap->seg0 + (size_t)rank * heap->L.stride + offset;
}

int symheap_reset(symheap_t *heap, void *cuda_stream)
{
    if (!heap) return SYMAR_ERR_INVAL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    CU(cudaMemsetAsync(heap->mem, 0, kCtlBytes, s));
    for (int q = 0; q < heap->P; ++q) {
        CU(cudaMemsetAsync(heap->seg0 + (size_t)q * heap->L.stride + heap->L.ll_off, 0,
                           heap->L.seg_bytes - heap->L.ll_off, s));
        CU(cudaMemsetAsync(heap->seg0 + (size_t)q * heap->L.stride + heap->L.sn_off, 0xff, heap->L.sn_bytes, s));
    }
    return SYMAR_OK;
}

int symheap_status(symheap_t *heap, int *code, int *rank, int *peer, int *cta)
{
    if (!heap) return SYMAR_ERR_INVAL;
    uint32_t w[4] = {0, 0, 0, 0};
    CU(cudaMemcpy(w, heap->ctl, sizeof w, cudaMemcpyDeviceToHost));
    if (code) *code = (int)w[kCtlCode];
    if (rank) *rank = (int)w[kCtlRank];
    if (peer) *peer = (int)w[kCtlPeer];
    if (cta) *cta = (int)w[kCtlCta];
    return SYMAR_OK;
}

int allreduce(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype,
              symar_algo_t algo, void *cuda_stream)
{
    return run(heap, in, out, count, (int)dtype, (int)algo, (cudaStream_t)cuda_stream);
}

// Host-buffer path for large messages: the message is cut into chunks; chunk i+1 travels to the
// device while chunk i is reduced and chunk i-1 travels back (the AllReduce is elementwise, so a
// chunk is an AllReduce of its own).  Both directions of the host link are busy at once.
constexpr size_t kHostChunkBytes = (size_t)16 << 20;      // per rank
constexpr int    kHostMaxChunks  = 64;

static int host_pipeline(symheap *h, const char *host_in, char *host_out, size_t io, size_t oo, size_t count, int dtype,
                         int algo, cudaStream_t s)
{
    const size_t es = elem_size(dtype), bytes = count * es;
    size_t chunk = kHostChunkBytes;
    while ((bytes + chunk - 1) / chunk > (size_t)kHostMaxChunks) chunk *= 2;
    const int n = (int)((bytes + chunk - 1) / chunk);
    if (!h->h2d) {
        CU(cudaStreamCreateWithFlags(&h->h2d, cudaStreamNonBlocking));
        CU(cudaStreamCreateWithFlags(&h->d2h, cudaStreamNonBlocking));
    }
    while (h->pipe_ev.size() < (size_t)(2 * kHostMaxChunks + 2)) {
        cudaEvent_t ev;
        CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
        h->pipe_ev.push_back(ev);
    }
    cudaEvent_t start = h->pipe_ev[0], end = h->pipe_ev[1];
    CU(cudaEventRecord(start, s));                          // everything enqueued so far comes first
    CU(cudaStreamWaitEvent(h->h2d, start, 0));
    for (int i = 0; i < n; ++i) {
        const size_t off = (size_t)i * chunk, len = std::min(chunk, bytes - off);
        for (int q = 0; q < h->P; ++q)
            CU(cudaMemcpyAsync(h->seg0 + (size_t)q * h->L.stride + io + off, host_in + (size_t)q * bytes + off, len,
                               cudaMemcpyHostToDevice, h->h2d));
        CU(cudaEventRecord(h->pipe_ev[2 + 2 * i], h->h2d));
    }
    for (int i = 0; i < n; ++i) {
        const size_t off = (size_t)i * chunk, len = std::min(chunk, bytes - off);
        CU(cudaStreamWaitEvent(s, h->pipe_ev[2 + 2 * i], 0));
        const int rc = run(h, h->seg0 + io + off, h->seg0 + oo + off, len / es, dtype, algo, s);
        if (rc != SYMAR_OK) return rc;
        CU(cudaEventRecord(h->pipe_ev[3 + 2 * i], s));
        CU(cudaStreamWaitEvent(h->d2h, h->pipe_ev[3 + 2 * i], 0));
        for (int r = 0; r < h->P; ++r)
            CU(cudaMemcpyAsync(host_out + (size_t)r * bytes + off, h->seg0 + (size_t)r * h->L.stride + oo + off, len,
                               cudaMemcpyDeviceToHost, h->d2h));
    }
    CU(cudaEventRecord(end, h->d2h));
    CU(cudaStreamWaitEvent(s, end, 0));                     // the caller's stream sees the results
    return SYMAR_OK;
}

int allreduce_host(symheap_t *heap, const void *host_in, void *host_out, const void *in, void *out,
                   size_t count, symar_dtype_t dtype, symar_algo_t algo, void *cuda_stream)
{
    size_t io = 0, oo = 0;
    int rc = check_buffers(heap, in, out, count, (int)dtype, &io, &oo);
    if (rc != SYMAR_OK) return rc;
    if (!host_in || !host_out) return SYMAR_ERR_INVAL;
    if ((int)algo < SYMAR_AUTO || (int)algo > kLastAlgo) return SYMAR_ERR_INVAL;
    if (count == 0) return SYMAR_OK;
    cudaStream_t s     = (cudaStream_t)cuda_stream;
    const size_t bytes = count * elem_size((int)dtype);
    if (bytes >= 2 * kHostChunkBytes && (io % 16 == 0) && (oo % 16 == 0))
        return host_pipeline(heap, (const char *)host_in, (char *)host_out, io, oo, count, (int)dtype, (int)algo, s);
    for (int q = 0; q < heap->P; ++q)
        CU(cudaMemcpyAsync(heap->seg0 + (size_t)q * heap->L.stride + io, (const char *)host_in + (size_t)q * bytes,
                           bytes, cudaMemcpyHostToDevice, s));
    rc = run(heap, in, out, count, (int)dtype, (int)algo, s);
    if (rc != SYMAR_OK) return rc;
    for (int r = 0; r < heap->P; ++r)
        CU(cudaMemcpyAsync((char *)host_out + (size_t)r * bytes, heap->seg0 + (size_t)r * heap->L.stride + oo,
                           bytes, cudaMemcpyDeviceToHost, s));
    return SYMAR_OK;
}

int symar_reduce_scatter(symheap_t *heap, const void *in, void *out, size_t recv_count, symar_dtype_t dtype,
                         void *cuda_stream)
{
    return run_collective(heap, 0, in, out, recv_count, (int)dtype, 0, (cudaStream_t)cuda_stream);
}

int symar_all_gather(symheap_t *heap, const void *in, void *out, size_t send_count, symar_dtype_t dtype,
                     void *cuda_stream)
{
    return run_collective(heap, 1, in, out, send_count, (int)dtype, 0, (cudaStream_t)cuda_stream);
}

int symar_broadcast(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype, int root,
                    void *cuda_stream)
{
    return run_collective(heap, 2, in, out, count, (int)dtype, root, (cudaStream_t)cuda_stream);
}

int symar_reduce(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype, int root,
                 void *cuda_stream)
{
    return run_collective(heap, 3, in, out, count, (int)dtype, root, (cudaStream_t)cuda_stream);
}

int allreduce_autotune(symheap_t *heap, symar_dtype_t dtype)
{
    if (!heap || (dtype != SYMAR_F32 && dtype != SYMAR_BF16)) return SYMAR_ERR_INVAL;
    return autotune(heap, (int)dtype, 0);
}

int allreduce_autotune_size(symheap_t *heap, symar_dtype_t dtype, size_t count)
{
    if (!heap || (dtype != SYMAR_F32 && dtype != SYMAR_BF16) || count == 0) return SYMAR_ERR_INVAL;
    if (count > heap->bytes_per_rank / elem_size((int)dtype)) return SYMAR_ERR_INVAL;
    return autotune(heap, (int)dtype, count * elem_size((int)dtype));
}

int allreduce_autotune_stream(symheap_t *heap, symar_dtype_t dtype, size_t count, int calls)
{
    if (!heap || (dtype != SYMAR_F32 && dtype != SYMAR_BF16) || count == 0 || calls < 2 || calls > 1024) return SYMAR_ERR_INVAL;
    const size_t es = elem_size((int)dtype);
    if (count > heap->bytes_per_rank / es) return SYMAR_ERR_INVAL;
    if (round_up(count * es, kAlign) * 2 * (size_t)calls > heap->bytes_per_rank) return SYMAR_ERR_INVAL;   // the pairs must fit
    return autotune(heap, (int)dtype, count * es, calls);
}

int symar_last_choice(const symheap_t *heap, symar_algo_t *algo, int *ctas_per_rank, int *threads)
{
    if (!heap) return SYMAR_ERR_INVAL;
    if (algo) *algo = (symar_algo_t)heap->last_algo;
    if (ctas_per_rank) *ctas_per_rank = heap->last_ctas;
    if (threads) *threads = heap->last_threads;
    return SYMAR_OK;
}

int symar_last_kernel(const symheap_t *heap, unsigned int *variant, size_t *shared_bytes)
{
    if (!heap) return SYMAR_ERR_INVAL;
    if (variant) *variant = heap->last_variant;
    if (shared_bytes) *shared_bytes = heap->last_smem;
    return SYMAR_OK;
}

int symar_query_choice(symheap_t *heap, size_t count, symar_dtype_t dtype, symar_algo_t *algo,
                       int *ctas_per_rank, int *threads)
{
    if (!heap || (dtype != SYMAR_F32 && dtype != SYMAR_BF16)) return SYMAR_ERR_INVAL;
    Plan p;
    int rc = make_plan(heap, 0, 0, count, (int)dtype, algo ? (int)*algo : SYMAR_AUTO, &p);
    if (rc != SYMAR_OK) return rc;
    if (algo) *algo = (symar_algo_t)p.algo;
    if (ctas_per_rank) *ctas_per_rank = p.cfg.ctas;
    if (threads) *threads = p.cfg.threads;
    return SYMAR_OK;
}

int symar_tuned_entry(const symheap_t *heap, symar_dtype_t dtype, int log2_bytes, symar_algo_t algo,
                      int *ctas_per_rank, int *threads, double *host_us)
{
    if (!heap || (dtype != SYMAR_F32 && dtype != SYMAR_BF16)) return SYMAR_ERR_INVAL;
    const Tuned &tn = heap->tuned[(int)dtype];
    if (log2_bytes < 0 || log2_bytes >= kBuckets) return SYMAR_ERR_INVAL;
    if (!tn.have[log2_bytes] && (!tn.valid || log2_bytes < tn.lo_bucket || log2_bytes > tn.hi_bucket))
        return SYMAR_ERR_INVAL;
    if (algo < SYMAR_ONESHOT || algo > kLastAlgo) return SYMAR_ERR_INVAL;
    if (ctas_per_rank) *ctas_per_rank = tn.cfg[algo][log2_bytes].ctas;
    if (threads) *threads = tn.cfg[algo][log2_bytes].threads;
    if (host_us) *host_us = tn.us[algo][log2_bytes];
    return SYMAR_OK;
}

// The tuned table as text: one header line, then per dtype and size bucket one "best"
// line and one line per algorithm.  Lets a deployment tune once per machine.
int symar_table_save(const symheap_t *heap, const char *host_path)
{
    if (!heap || !host_path) return SYMAR_ERR_INVAL;
    FILE *f = std::fopen(host_path, "w");
    if (!f) return SYMAR_ERR_INVAL;
    std::fprintf(f, "symar-table 1 P %d\n", heap->P);
    for (int dt = 0; dt < 2; ++dt) {
        const Tuned &tn = heap->tuned[dt];
        bool any = tn.valid;
        for (int b = 0; b < kBuckets; ++b) any = any || tn.have[b];
        if (!any) continue;
        // "buckets 0 -1": no grid, only buckets tuned one at a time ("have" lines)
        std::fprintf(f, "dtype %d buckets %d %d\n", dt, tn.valid ? tn.lo_bucket : 0, tn.valid ? tn.hi_bucket : -1);
        for (int b = 0; b < kBuckets; ++b) {
            const bool in_grid = tn.valid && b >= tn.lo_bucket && b <= tn.hi_bucket;
            if (!in_grid && !tn.have[b]) continue;
            if (tn.have[b]) std::fprintf(f, "have %d\n", b);
            std::fprintf(f, "best %d %d\n", b, tn.best_algo[b]);
            for (int a = SYMAR_ONESHOT; a < kAlgos; ++a)
                std::fprintf(f, "cfg %d %d %d %d %d %.6g\n", b, a, tn.cfg[a][b].ctas, tn.cfg[a][b].threads,
                             tn.cfg[a][b].variant, tn.us[a][b]);
        }
    }
    return std::fclose(f) == 0 ? SYMAR_OK : SYMAR_ERR_INVAL;
}

int symar_table_load(symheap_t *heap, const char *host_path)
{
    if (!heap || !host_path) return SYMAR_ERR_INVAL;
    FILE *f = std::fopen(host_path, "r");
    if (!f) return SYMAR_ERR_INVAL;
    int version = 0, P = 0;
    if (std::fscanf(f, "symar-table %d P %d", &version, &P) != 2 || version != 1 || P != heap->P) {
        std::fclose(f);
        return SYMAR_ERR_INVAL;          // written for another rank count or format
    }
    Tuned loaded[2];
    bool seen[2] = {false, false};
    int dt = -1;
    char word[16];
    bool ok = true;
    while (ok && std::fscanf(f, "%15s", word) == 1) {
        const std::string w(word);
        if (w == "dtype") {
            int lo, hi;
            ok = std::fscanf(f, "%d buckets %d %d", &dt, &lo, &hi) == 3 && dt >= 0 && dt < 2 && lo >= 0 &&
                 hi < kBuckets && (lo <= hi || (lo == 0 && hi == -1));
            if (ok) {
                loaded[dt]           = Tuned{};
                loaded[dt].lo_bucket = lo;
                loaded[dt].hi_bucket = hi;
                loaded[dt].valid     = lo <= hi;
                seen[dt]             = true;
                for (int b = 0; b < kBuckets; ++b) {
                    loaded[dt].best_algo[b] = SYMAR_ONESHOT;
                    for (int a = 0; a < kAlgos; ++a) loaded[dt].us[a][b] = 1e30;
                }
            }
        } else if (w == "have") {
            int b;
            ok = dt >= 0 && std::fscanf(f, "%d", &b) == 1 && b >= 0 && b < kBuckets;
            if (ok) loaded[dt].have[b] = true;
        } else if (w == "best") {
            int b, a;
            ok = dt >= 0 && std::fscanf(f, "%d %d", &b, &a) == 2 && b >= 0 && b < kBuckets && a >= SYMAR_ONESHOT &&
                 a < kAlgos;
            if (ok) loaded[dt].best_algo[b] = a;
        } else if (w == "cfg") {
            int b, a, c, t, v;
            double us;
            ok = dt >= 0 && std::fscanf(f, "%d %d %d %d %d %lf", &b, &a, &c, &t, &v, &us) == 6 && b >= 0 &&
                 b < kBuckets && a >= SYMAR_ONESHOT && a < kAlgos && c >= 0 && c <= kMaxCtas && t >= 0 &&
                 t <= (int)kMaxThreads;
            if (ok) {
                loaded[dt].cfg[a][b] = LaunchCfg{c, t, v};
                loaded[dt].us[a][b]  = us;
            }
        } else {
            ok = false;
        }
    }
    std::fclose(f);
    if (!ok) return SYMAR_ERR_INVAL;
    for (int d = 0; d < 2; ++d)
        if (seen[d]) heap->tuned[d] = loaded[d];
    return SYMAR_OK;
}

int symar_set_launch(symheap_t *heap, symar_algo_t algo, int ctas_per_rank, int threads)
{
    if (!heap || algo < SYMAR_ONESHOT || algo > kLastAlgo) return SYMAR_ERR_INVAL;
    if (ctas_per_rank < 0 || threads < 0 || threads > (int)kMaxThreads) return SYMAR_ERR_INVAL;
    heap->forced[algo] = LaunchCfg{ctas_per_rank, threads};
    return SYMAR_OK;
}

int symar_set_variant(symheap_t *heap, symar_algo_t algo, unsigned int variant)
{
    if (!heap || algo < SYMAR_ONESHOT || algo > kLastAlgo) return SYMAR_ERR_INVAL;
    heap->variant[algo]        = variant & 0x7fffffffu;
    heap->variant_forced[algo] = variant != 0;       // bit 31 alone forces the plain variant 0
    return SYMAR_OK;
}

int symar_set_pdl(symheap_t *heap, int enabled)
{
    if (!heap) return SYMAR_ERR_INVAL;
    heap->pdl = enabled != 0;
    return SYMAR_OK;
}

int symar_set_placement(symheap_t *heap, int enabled)
{
    if (!heap) return SYMAR_ERR_INVAL;
    heap->place_on = enabled != 0;
    return SYMAR_OK;
}

int symar_placement(const symheap_t *heap, int *measured, int *sms_on_half1, unsigned long long *home_bits)
{
    if (!heap) return SYMAR_ERR_INVAL;
    if (measured) *measured = heap->placed ? 1 : 0;
    if (sms_on_half1) {
        int n = 0;
        for (int i = 0; i < 4; ++i) n += __builtin_popcountll(heap->sm_half[i]);
        *sms_on_half1 = n;
    }
    if (home_bits) *home_bits = heap->home;
    return SYMAR_OK;
}

int symar_set_scratch_limit(symheap_t *heap, size_t payload_bytes_per_iteration)
{
    if (!heap) return SYMAR_ERR_INVAL;
    heap->scratch_limit = payload_bytes_per_iteration;
    return SYMAR_OK;
}

int symar_set_spin_limit_us(symheap_t *heap, unsigned int microseconds)
{
    if (!heap || microseconds == 0) return SYMAR_ERR_INVAL;
    heap->spin_ns = (uint64_t)microseconds * 1000ull;
    return SYMAR_OK;
}

int symar_debug_inject(symheap_t *heap, int mute_rank, unsigned int delay_seed, unsigned int delay_max_ns)
{
    if (!heap || mute_rank >= heap->P) return SYMAR_ERR_INVAL;
    if (delay_max_ns > 1000000u) return SYMAR_ERR_INVAL;   // keep test delays below a millisecond
    heap->dbg_mute     = mute_rank < 0 ? -1 : mute_rank;
    heap->dbg_seed     = delay_seed;
    heap->dbg_delay_ns = delay_max_ns;
    return SYMAR_OK;
}

const char *symar_last_cuda_error(void) { return g_last_cuda_error.c_str(); }

int symar_debug_span(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype,
                     symar_algo_t algo, void *cuda_stream, double *host_span_ns)
{
    if (!heap || !host_span_ns) return SYMAR_ERR_INVAL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const unsigned long long init[2] = {~0ull, 0ull};
    CU(cudaMemcpyAsync(heap->ctl + kCtlSpanIn, init, sizeof init, cudaMemcpyHostToDevice, s));
    CU(cudaStreamSynchronize(s));                       // `init` is on this stack frame
    heap->dbg_span = true;
    const int rc = run(heap, in, out, count, (int)dtype, (int)algo, s);
    heap->dbg_span = false;
    if (rc != SYMAR_OK) return rc;
    unsigned long long w[2] = {0, 0};
    CU(cudaMemcpyAsync(w, heap->ctl + kCtlSpanIn, sizeof w, cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    if (w[0] == ~0ull || w[1] < w[0]) return SYMAR_ERR_UNSUPPORTED;     // this kernel carries no stamps
    *host_span_ns = (double)(w[1] - w[0]);
    return SYMAR_OK;
}

int symar_debug_phases(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype,
                       symar_algo_t algo, void *cuda_stream, double *host_ns, int *host_stamps)
{
    if (!heap || !host_ns || !host_stamps) return SYMAR_ERR_INVAL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    unsigned long long w[4 * kPhases];
    for (int k = 0; k < kPhases; ++k) {
        w[k]               = ~0ull;     // earliest
        w[kPhases + k]     = 0ull;      // latest
        w[2 * kPhases + k] = 0ull;      // wrapping sum
        w[3 * kPhases + k] = 0ull;      // stamps
    }
    CU(cudaMemcpyAsync(heap->ctl + kCtlPhaseMin, w, sizeof w, cudaMemcpyHostToDevice, s));
    CU(cudaStreamSynchronize(s));                       // `w` is on this stack frame
    heap->dbg_span = true;
    const int rc = run(heap, in, out, count, (int)dtype, (int)algo, s);
    heap->dbg_span = false;
    if (rc != SYMAR_OK) return rc;
    CU(cudaMemcpyAsync(w, heap->ctl + kCtlPhaseMin, sizeof w, cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    if (w[3 * kPhases] == 0) return SYMAR_ERR_UNSUPPORTED;             // this kernel carries no stamps
    const unsigned long long t0 = w[0];
    for (int k = 0; k < kPhases; ++k) {
        const unsigned long long n = w[3 * kPhases + k];
        host_stamps[k] = (int)n;
        if (n == 0) {
            host_ns[3 * k] = host_ns[3 * k + 1] = host_ns[3 * k + 2] = -1.0;
            continue;
        }
        host_ns[3 * k]     = (double)(long long)(w[k] - t0);
        host_ns[3 * k + 1] = (double)(long long)(w[2 * kPhases + k] - n * t0) / (double)n;   // sums wrap; the difference does not
        host_ns[3 * k + 2] = (double)(long long)(w[kPhases + k] - t0);
    }
    return SYMAR_OK;
}

int symar_check_selftest(symheap_t *heap, void *cuda_stream)
{
    if (!heap || heap->bytes_per_rank < 4096) return SYMAR_ERR_INVAL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    Plan p;
    int rc = make_plan(heap, 0, 1024, 16, SYMAR_F32, SYMAR_ONESHOT, &p);      // a 64-byte call: in at 0, out at 1024
    if (rc != SYMAR_OK) return rc;
    const uint32_t before[4] = {0xAAAAAAAAu, 0xAAAAAAAAu, 0xAAAAAAAAu, 0xAAAAAAAAu};
    CU(cudaMemcpyAsync(heap->seg0 + 1024 + 64, before, sizeof before, cudaMemcpyHostToDevice, s));
    CU(cudaStreamSynchronize(s));                          // `before` is on this stack frame
    cudaError_t e = launch_check_selftest(p.args, s);
    if (e == cudaErrorNotSupported) {
        cudaGetLastError();
        return SYMAR_ERR_UNSUPPORTED;                      // the regular build checks nothing
    }
    if (e != cudaSuccess) return cuda_fail(e, "self-test launch");
    uint32_t inside[4] = {0, 0, 0, 0}, beyond[4] = {0, 0, 0, 0}, status[4] = {0, 0, 0, 0};
    CU(cudaMemcpyAsync(inside, heap->seg0 + 1024, sizeof inside, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(beyond, heap->seg0 + 1024 + 64, sizeof beyond, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(status, heap->ctl, sizeof status, cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    const bool landed  = inside[0] == 1u && inside[3] == 4u;
    const bool kept    = std::memcmp(beyond, before, sizeof before) == 0;
    const bool flagged = (int)status[kCtlCode] == SYMAR_ERR_INVAL && status[kCtlPeer] == (uint32_t)kRegOutMask;
    CU(cudaMemsetAsync(heap->ctl, 0, 16, s));              // the recorded violation was the point: clear it
    CU(cudaStreamSynchronize(s));
    return (landed && kept && flagged) ? SYMAR_OK : SYMAR_ERR_CUDA;
}

size_t symar_llbuffer_bytes(int sync_mode, size_t elem_bytes, size_t slots_per_cta, int ctas, int round_robin)
{
    if ((sync_mode != 0 && sync_mode != 1) || (elem_bytes != 4 && elem_bytes != 8) || ctas < 1 || round_robin < 0)
        return 0;
    return (sync_mode == 0 ? 2 : 1) * elem_bytes * slots_per_cta * (size_t)ctas * (size_t)(round_robin ? round_robin : 1);
}

int symar_llbuffer_init_sentinel(void *device_ptr, size_t bytes, void *cuda_stream)
{
    if (!device_ptr) return SYMAR_ERR_INVAL;
    CU(cudaMemsetAsync(device_ptr, 0xff, bytes, (cudaStream_t)cuda_stream));
    return SYMAR_OK;
}

}  // extern "C"
