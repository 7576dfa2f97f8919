/*
 * symar -- barrier-free symmetric-memory AllReduce(sum) for one B200.
 *
 * C ABI of libsymar.so.  Plain pointers and sizes only; no C++ or framework
 * types cross this boundary.  Unless a parameter says "host", a pointer is a
 * DEVICE address.
 *
 * Model.  P ranks are emulated on one GPU as disjoint CTA partitions of ONE
 * kernel launch.  They share a symmetric heap (paper Sec. II-B: every rank holds
 * an object of the same type, size and layout at the same offset):
 * P equally laid-out rank segments, so that the object at byte offset `o` of
 * rank q is always  base + q * stride + o.  Ranks meet only through that memory,
 * exactly as GPUs of one NVLink domain meet through load/store-accessible
 * peer memory.  Synchronisation never uses a grid-wide or memory barrier
 * (Sec. III-B): one-shot and two-shot use per-peer sequence-number flags, the
 * LL protocol carries a flag inside every 8-byte store (Sec. IV "LL").
 *
 * Every function returns an int status: SYMAR_OK (0) or a negative error.
 * Nothing throws, aborts or prints.  All device-side waits are bounded; a wait
 * that gives up records SYMAR_ERR_TIMEOUT in the heap's status word (read it
 * with symheap_status) and the kernel returns normally.
 *
 * Environment (read when a heap is created): SYMAR_ALGO = oneshot | twoshot | ll |
 * sentinel | twoshot_ll | twoshot_sentinel | twoshot_atomic replaces SYMAR_AUTO's choice;
 * SYMAR_CTAS_PER_RANK and SYMAR_THREADS fix the launch shape of every algorithm;
 * SYMAR_SPIN_LIMIT_US bounds device-side waits; SYMAR_PDL = 0 turns programmatic dependent
 * launch off; SYMAR_DEBUG = 1 logs every call's resolved algorithm and shape to stderr
 * (nothing is printed otherwise); SYMAR_TUNE = exhaustive makes allreduce_autotune time every
 * algorithm and shape at every size instead of pruning by the previous size's result;
 * SYMAR_PLACE = 0 turns the placement of flag and counter reads on the chip's L2 halves off;
 * SYMAR_CLUSTER = 0 keeps every launch a plain one (see SYMAR_VARIANT_CLUSTER).
 *
 * Threading: a heap may be used from one host thread and one stream at a time
 * (the per-CTA epoch counters live in the heap).  Calls on one stream are
 * ordered by the stream.
 *
 * What a call needs from the GPU: the CTAs of the P ranks wait for one another, so
 * all P x C CTAs of a launch must be resident at the same time.  The library sizes
 * every launch to what fits on the IDLE device; it cannot see other work.  Kernels
 * of other streams or processes that hold SMs while a call runs (a second heap, a
 * compute kernel of the caller, allreduce_static next to a heap call) can keep part
 * of the grid from starting; the resident CTAs then wait until the bound expires
 * (default 0.2 s), the call reports SYMAR_ERR_TIMEOUT and `out` is undefined.  Give
 * the collective the device for its few microseconds: order it after the work
 * before it on one stream, as a tensor-parallel layer does anyway.
 */
#ifndef SYMAR_H
#define SYMAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct symheap symheap_t;            /* opaque; owned by the library */

typedef enum { SYMAR_F32 = 0, SYMAR_BF16 = 1 } symar_dtype_t;

typedef enum {
    SYMAR_AUTO    = 0,   /* per-size selector (Sec. VIII: the fastest low-latency algorithm for
                            a size is chosen from measurements taken beforehand)              */
    SYMAR_ONESHOT = 1,   /* Sec. III-A.1, pull form: every rank reads all P inputs           */
    SYMAR_TWOSHOT = 2,   /* Sec. III-A.2: reduce-scatter, then all-gather with flag handoff  */
    SYMAR_LL      = 3,   /* Sec. IV "LL" + Sec. V example: one-shot push, data+flag stores   */
    SYMAR_SENTINEL = 4,  /* Sec. IV "Sentinel": one-shot push of bare data into scratch that
                            holds a sentinel word; the receiver polls until every word has
                            changed and restores the sentinel.                               */
    SYMAR_TWOSHOT_LL = 5,       /* Table I "Two-shot (LL)": reduce-scatter and all-gather both
                                   pushed through the LL scratch, synchronised by the data    */
    SYMAR_TWOSHOT_SENTINEL = 6, /* Table I "Two-shot (Sentinel)": the same through the sentinel
                                   scratch.  (SYMAR_AUTO picks algorithms 3..6 only where the
                                   tuner measured them to be fastest.)                        */
    SYMAR_TWOSHOT_ATOMIC = 7    /* Sec. IV "LL128 Atomic AllReduce" / Table I last row: every rank
                                   ADDS its part of chunk t into rank t's scratch with 16-byte
                                   vector atomics; a contribution counter rides in each 128-byte
                                   line; the owner polls it, then stores the sums everywhere.
                                   NOT bit-reproducible (the order of the binary32 atomic adds is
                                   free): results stay within gamma_{P-1} * sum|x_q| of the exact
                                   sum; subnormals are flushed by the atomics.  bf16 is
                                   accumulated in binary32 and narrowed once.  One call reduces
                                   at most 31 * 4096 * P * P elements (SYMAR_ERR_UNSUPPORTED
                                   above).  Never chosen by SYMAR_AUTO or the tuner.           */
} symar_algo_t;

enum {
    SYMAR_OK              =  0,
    SYMAR_ERR_INVAL       = -1,   /* bad argument (null, misaligned, out of range, overlap)  */
    SYMAR_ERR_NOMEM       = -2,   /* device or host allocation failed / caller memory too small */
    SYMAR_ERR_CUDA        = -3,   /* a CUDA runtime call failed; see symar_last_cuda_error()  */
    SYMAR_ERR_TIMEOUT     = -4,   /* a bounded device-side wait gave up (via symheap_status)  */
    SYMAR_ERR_UNSUPPORTED = -5    /* valid request this build cannot serve                    */
};

/* Compile-time shape of a rank segment (all sizes in bytes unless noted). */
enum {
    SYMAR_MAX_RANKS     = 8,      /* P must be 1, 2, 4 or 8                                   */
    SYMAR_MAX_CTAS      = 160,    /* CTA slots per rank that own flags and an epoch counter   */
    SYMAR_LL_SLOTS      = 64,     /* CTA slots per rank that own an LL scratch region          */
    SYMAR_LL_SLOT_VECS  = 1024,   /* 16-byte payload vectors per LL slot, sender and iteration */
    SYMAR_ALIGN         = 8192    /* alignment of the heap and of every region of a segment:
                                     streams that start on 1 KiB boundaries use HBM best, and
                                     flags and counters live in 8 KiB pairs of 4 KiB copies,
                                     one copy per half of the chip's L2                         */
};

typedef struct {
    int      P;                   /* ranks                                                     */
    size_t   bytes_per_rank;      /* user region as requested                                   */
    size_t   user_bytes;          /* user region as laid out (rounded up to SYMAR_ALIGN)        */
    size_t   ll_scratch_bytes;    /* per rank: 2 parities x slots x P senders x vecs x 32 B     */
    size_t   sentinel_scratch_bytes; /* per rank: 2 parities x slots x P senders x vecs x 16 B   */
    size_t   atomic_scratch_bytes; /* per rank: 2 parities x 512 KiB x P of 128-byte lines     */
    size_t   flag_bytes;          /* per rank: ready + done flag arrays + counters, two copies of each */
    size_t   stride;              /* bytes from one rank segment to the next                    */
    size_t   total_bytes;         /* control block + P segments                                 */
    void    *base;                /* device address of rank 0's segment                         */
} symheap_info_t;

/* ---- symmetric heap (Sec. II-B symmetric heap; Sec. IV scratch buffer; Sec. V
 *      ncclLLBuffer layout "address = f(epoch, CTA index)") ------------------- */

/* Bytes of device memory a heap of P ranks with `bytes_per_rank` of user region
 * needs (control block + P segments of user region, LL, sentinel and atomic
 * scratch, flags and counters).
 * Returns 0 if P is not 1, 2, 4 or 8.                                          */
size_t symheap_required_bytes(int P, size_t bytes_per_rank);

/* Create a heap in memory the library allocates with cudaMalloc on the current
 * device and frees in symheap_destroy.  Scratch and flags are zeroed
 * (synchronously).  *heap is written only on success.                          */
int symheap_create(symheap_t **heap, int P, size_t bytes_per_rank);

/* As symheap_create, in caller-owned device memory (e.g. a torch tensor) of at
 * least symheap_required_bytes() bytes, SYMAR_ALIGN-byte aligned.  The caller keeps the
 * memory alive until symheap_destroy and frees it afterwards.                  */
int symheap_create_on(symheap_t **heap, int P, size_t bytes_per_rank,
                      void *device_mem, size_t device_bytes);

int symheap_destroy(symheap_t *heap);

/* Layout of the heap (host struct filled in). */
int symheap_info(const symheap_t *heap, symheap_info_t *info);

/* Device address of byte `offset` of rank `rank`'s user region; NULL when out
 * of range.  symheap_rank_ptr(h, 0, o) is the "symmetric address" that
 * allreduce() takes for the object at offset o of every rank.                  */
void *symheap_rank_ptr(const symheap_t *heap, int rank, size_t offset);

/* Zero scratch, flags, epoch counters and the status word (asynchronous on
 * `cuda_stream`).  Needed only after a SYMAR_ERR_TIMEOUT left them inconsistent. */
int symheap_reset(symheap_t *heap, void *cuda_stream);

/* Synchronous read of the device status word: *code is SYMAR_OK or
 * SYMAR_ERR_TIMEOUT; on timeout *rank / *peer / *cta say which emulated rank's
 * CTA slot gave up waiting for which peer.  Any out pointer may be NULL.       */
int symheap_status(symheap_t *heap, int *code, int *rank, int *peer, int *cta);

/* ---- the collective ---------------------------------------------------------
 *
 * out[r][i] = narrow( ((x_0[i] + x_1[i]) + ... ) + x_{P-1}[i] )   for every rank r,
 * x_q = widen(in[q]), sum in IEEE binary32 in rank order 0..P-1 (the deterministic
 * one-/two-shot rows of Table I; accumulator type per Sec. V recvReduce), bf16
 * narrowed once with round-to-nearest-even.  Every algorithm gives these bits, except
 * SYMAR_TWOSHOT_ATOMIC, whose order of additions is free (see its enumerator).
 *
 * in, out : symmetric addresses -- device pointers into RANK 0's user region
 *           (symheap_rank_ptr(heap, 0, off)); rank q's buffer is the same offset
 *           in its own segment.  16-byte aligned (1 KiB-aligned buffers stream
 *           fastest for large messages).  Out-of-place only (Sec. VII
 *           measures out-of-place): the byte ranges must not overlap.
 * count   : elements PER RANK.  0 is a no-op.  Any count is accepted; a ragged
 *           tail is handled inside the kernels.
 * algo    : SYMAR_AUTO picks by table lookup (no timing at call time).  A named
 *           algorithm is never silently replaced.
 * cuda_stream : cudaStream_t (NULL = legacy default stream).  The call enqueues
 *           exactly one kernel and returns; it may be captured in a CUDA graph.
 * Errors  : SYMAR_ERR_INVAL for a bad pointer/alignment/range/overlap/dtype/algo;
 *           SYMAR_ERR_CUDA if the launch failed.                                */
int allreduce(symheap_t *heap, const void *in, void *out, size_t count,
              symar_dtype_t dtype, symar_algo_t algo, void *cuda_stream);

/* The same collective for HOST buffers (end-to-end path): copies row q of
 * host_in ([P][count] elements, row-major, host memory, ideally pinned) to rank
 * q's `in`, runs allreduce(), copies every rank's `out` to row r of host_out
 * ([P][count]).  Ordered on `cuda_stream` like any other call; the host buffers
 * must stay valid until the stream has drained.  Messages of 32 MiB per rank and
 * more are cut into 16 MiB chunks (an elementwise sum is a sum of its chunks) that
 * move on two copy streams of the heap, so that chunk i+1 travels to the device
 * while chunk i is reduced and chunk i-1 travels back: one kernel per chunk, both
 * directions of the host link busy at once.  The algorithm is resolved per chunk. */
int allreduce_host(symheap_t *heap, const void *host_in, void *host_out,
                   const void *in, void *out, size_t count,
                   symar_dtype_t dtype, symar_algo_t algo, void *cuda_stream);

/* ---- sibling collectives (Sec. V "NCCL Collective Integration": Broadcast, Reduce,
 *      ReduceScatter and AllGather from the same primitives; Sec. III: AllReduce =
 *      ReduceScatter + AllGather = Reduce + Broadcast) ----------------------------
 *
 * Same conventions as allreduce(): symmetric addresses, 16-byte aligned, out-of-place,
 * one kernel per call on `cuda_stream`, one signal exchange, bounded waits.  Sums are
 * the rank-ordered binary32 sum with one narrowing.  Every rank writes only its own
 * output.
 *   symar_reduce_scatter  in: P * recv_count elements per rank; rank r's out (recv_count
 *                         elements) = sum over q of in[q][r * recv_count ...]
 *   symar_all_gather      in: send_count elements per rank; every rank's out holds the
 *                         P inputs back to back (P * send_count elements)
 *   symar_broadcast       every rank's out = rank `root`'s in (count elements)
 *   symar_reduce          rank `root`'s out = the sum of all ranks' in; other ranks' out
 *                         is left untouched                                              */
int symar_reduce_scatter(symheap_t *heap, const void *in, void *out, size_t recv_count,
                         symar_dtype_t dtype, void *cuda_stream);
int symar_all_gather(symheap_t *heap, const void *in, void *out, size_t send_count,
                     symar_dtype_t dtype, void *cuda_stream);
int symar_broadcast(symheap_t *heap, const void *in, void *out, size_t count,
                    symar_dtype_t dtype, int root, void *cuda_stream);
int symar_reduce(symheap_t *heap, const void *in, void *out, size_t count,
                 symar_dtype_t dtype, int root, void *cuda_stream);

/* ---- selector (Sec. VIII kernel selection; Sec. IX: selection is empirical) --
 *
 * Times the algorithms and their launch shapes over a power-of-two grid of message
 * sizes (16 B ... min(bytes_per_rank / 2, 64 MiB) per rank) on an internal
 * stream, and fills the (P, dtype) table that SYMAR_AUTO and the default launch
 * shapes consult.  Going up the grid, an algorithm that moves more bytes than the
 * winner and lost by more than 1.5 x one size down is not timed again, and shapes
 * are searched around the previous size's winner (SYMAR_TUNE = exhaustive in the
 * environment searches everything).  Synchronous; takes seconds.  OVERWRITES the
 * user region of every rank.  Before it is called, built-in defaults apply: the
 * data+flag protocol up to 128 KiB between two ranks, 32 KiB among four and 256 B among eight, else one-shot up to
 * 256 KiB x (8 / P)^2 per rank, else two-shot, each in a launch shape that restates
 * what this tuner chose on B200 (within a few percent of a tuned call).          */
int allreduce_autotune(symheap_t *heap, symar_dtype_t dtype);

/* The same for ONE message size: times every algorithm, shape and variant on messages
 * of exactly `count` elements per rank (2 * count elements must fit in the user region)
 * and records the winners for that size's bucket only, next to whatever the table
 * already holds.  A second or two even for hundreds of MiB; for deployments that know
 * their message sizes, and for sizes beyond the 64 MiB grid.  OVERWRITES the user region. */
int allreduce_autotune_size(symheap_t *heap, symar_dtype_t dtype, size_t count);

/* The same for one message size as it occurs in a STREAM of calls that each have their own buffers
 * (the AllReduces of a decode step: 2 per layer, every one on activations that were just produced):
 * every candidate is timed in a graph of `calls` (2..1024) back-to-back calls, call k on the k-th of
 * `calls` input / output pairs laid side by side in the user region (2 * calls * count elements,
 * rounded up to SYMAR_ALIGN per buffer, must fit).  With enough pairs the inputs are not in L2 when
 * a call starts, and the shape that is best then is not always the one that is best on warm buffers.
 * Records the winners for that size's bucket only.  OVERWRITES the user region.                 */
int allreduce_autotune_stream(symheap_t *heap, symar_dtype_t dtype, size_t count, int calls);

/* What the last allreduce() on this heap launched (for reporting). */
int symar_last_choice(const symheap_t *heap, symar_algo_t *algo,
                      int *ctas_per_rank, int *threads);

/* Kernel variant bits (see symar_set_variant) and dynamic shared memory of the
 * last launch; shared_bytes > 0 means the bulk-copy two-shot kernel ran.          */
int symar_last_kernel(const symheap_t *heap, unsigned int *variant, size_t *shared_bytes);

/* What SYMAR_AUTO would launch for a message of `count` elements. */
int symar_query_choice(symheap_t *heap, size_t count, symar_dtype_t dtype,
                       symar_algo_t *algo, int *ctas_per_rank, int *threads);

/* One row of the table allreduce_autotune() filled: for messages of 2^log2_bytes
 * bytes per rank, the best launch shape found for `algo` and its measured time
 * per call in microseconds (host double).  SYMAR_ERR_INVAL if not tuned.       */
int symar_tuned_entry(const symheap_t *heap, symar_dtype_t dtype, int log2_bytes,
                      symar_algo_t algo, int *ctas_per_rank, int *threads, double *host_us);

/* Write / read the tuned table as a small text file (host path), so that a
 * deployment tunes once per machine.  Loading rejects a file written for another
 * rank count or with out-of-range entries (SYMAR_ERR_INVAL); launch shapes are
 * re-clamped to what is co-resident at call time in any case.                   */
int symar_table_save(const symheap_t *heap, const char *host_path);
int symar_table_load(symheap_t *heap, const char *host_path);

/* Force the launch shape of one algorithm (0 = back to table/default).  The
 * library still clamps P * ctas_per_rank to what is co-resident on the device:
 * CTAs of different ranks wait for one another, so all must be resident.       */
int symar_set_launch(symheap_t *heap, symar_algo_t algo, int ctas_per_rank, int threads);

/* Implementation variant of one algorithm's kernel, for performance experiments;
 * every variant computes the same bits.  0 = back to the table/default choice;
 * bit 31 alone forces the plain variant (all other bits 0).  One-shot: bits 8-9 = bytes
 * per thread (0: 16, 1: 8, 2: 4), bit 14 = the prior-art form with a memory-ordering barrier
 * before the data phase and another before returning (what Sec. III-B removes; for comparison),
 * bit 15 = release ordering on the "input ready" signal and nothing else changed (what the
 * exchange costs where no kernel boundary publishes the inputs; for comparison).  LL: bit 8 = 8
 * instead of 16 payload bytes per thread, bit 9 = the general (looping) kernel even where the
 * single-iteration kernel covers the message, bits 12-15 = cycles / 64 by which the
 * single-iteration kernel holds back its first poll;
 * two-shot: bit 0 = contiguous chunks also for large messages (no block-cyclic
 * ownership), bit 1 = 16-byte instead of 32-byte accesses for large messages,
 * bit 2 = the register kernel instead of the bulk-copy kernel from 4 MiB (the built-in
 * choice there), bit 6 = 8 instead of 16 bytes per thread and
 * trip for messages below 1 MiB, bits 8-10 = the bulk kernel's pipeline depth (0:
 * default), bits 12-13 = log2 of its tile size over 4 KiB.
 * Every algorithm: SYMAR_VARIANT_CLUSTER (bit 30) = the P CTAs of a slot, one per rank, are launched
 * as one thread-block cluster, i.e. on SMs of one GPC and so on one half of the chip.  Only their
 * placement changes: the kernels use nothing of a cluster (no distributed shared memory, no cluster
 * barrier), the ranks meet through flags in global memory as before.  Ignored for one rank and for the
 * bulk-copy kernel; where the clusters of a shape cannot all be resident, that shape is launched
 * plainly (symar_last_kernel tells).  The built-in choice and the tuner set it where it was measured
 * faster: the data+flag protocol at every size, the others while their CTAs are few.              */
#define SYMAR_VARIANT_CLUSTER 0x40000000u
int symar_set_variant(symheap_t *heap, symar_algo_t algo, unsigned int variant);

/* Programmatic dependent launch (ON by default; SYMAR_PDL=0 in the environment or
 * enabled = 0 here turns it off).  When on, every kernel of the library is launched
 * so that it may become resident while the previous kernel of the stream still runs;
 * its first instruction waits until that grid has completed and its writes are
 * visible, so results and ordering are unchanged -- only the launch latency of
 * back-to-back calls is hidden (measured: -0.25 us of 1.95 us per 16 KiB call).  */
int symar_set_pdl(symheap_t *heap, int enabled);

/* Placement on the chip's two L2 halves (ON by default; SYMAR_PLACE=0 in the environment at heap
 * creation, or enabled = 0 here, turns it off).  B200's L2 is two halves; a line that has just been
 * written is read about twice as fast from an SM on the half that homes it.  A heap keeps two copies of
 * every flag and counter, homed on opposite halves (addresses that differ in bit 12 only); writers update
 * both, and with placement on a reader takes the copy of its own SM's half, as measured when the heap
 * was created (which half each SM sits on; which half homes which copy).  Off, or if that measurement
 * was not clean, every reader takes copy 0.  Results are the same bits either way.
 * symar_placement reports: *measured = 1 if the measurement was clean, *sms_on_half1 = SMs found on the
 * second half, *home_bits = per rank one byte, bit p = half that homes copy 0 of the rank's pair p
 * (ready flags 0-1, done flags 2-3, counters 4).  Out pointers may be NULL.                        */
int symar_set_placement(symheap_t *heap, int enabled);
int symar_placement(const symheap_t *heap, int *measured, int *sms_on_half1, unsigned long long *home_bits);

/* Pretend the push algorithms (LL, sentinel, and their two-shot forms) had a smaller
 * scratch buffer: at most `payload_bytes_per_iteration` bytes of each rank's message are
 * reduced per iteration (Table I's D), so larger messages take more iterations, each
 * with its own synchronisation (Sec. VII "Impact of Scratch Buffer").  0 = use all of
 * the scratch (1 MiB of payload per rank and iteration for the one-shot forms).       */
int symar_set_scratch_limit(symheap_t *heap, size_t payload_bytes_per_iteration);

/* Upper bound of any device-side wait, in microseconds.  Default 200 000 (0.2 s: hundreds of
 * times the longest call, and short enough not to hold a shared GPU when a wait can never end);
 * SYMAR_SPIN_LIMIT_US in the environment or this call change it.                      */
int symar_set_spin_limit_us(symheap_t *heap, unsigned int microseconds);

/* Test hooks; all off by default and free when off (separate kernel
 * instantiation).  delay_max_ns > 0: every CTA first idles for a seeded
 * pseudo-random time below delay_max_ns, to vary the interleaving of ranks.
 * mute_rank >= 0: that rank sends no data and raises no flags, so that its
 * peers' bounded waits run out (exercises SYMAR_ERR_TIMEOUT without a fault).  */
int symar_debug_inject(symheap_t *heap, int mute_rank, unsigned int delay_seed,
                       unsigned int delay_max_ns);

/* ---- AllReduce without any allocation ------------------------------------------
 *
 * (The paper has no counterpart of this entry point: its kernels take their
 * scratch from NCCL's symmetric-memory allocator.)
 *
 * For callers that cannot allocate device memory -- code running with a frozen
 * memory pool inside a serving loop, a plugin that was handed no allocator, code
 * that may run while another thread captures a CUDA graph (an allocation would
 * break the capture), or a deployment that fixes all device memory at start-up --
 * and therefore cannot create a symmetric heap.  The caller passes plain device
 * buffers; the LL protocol's scratch and its counters live in one file-scope
 * __device__ array of about 8 MiB that every GPU which loads the library holds
 * until the process exits.  This function and everything it calls allocate and
 * free nothing (no cudaMalloc/cudaFree, no allocating library routine).
 *
 * in, out : device buffers of P rows; rank q's input is at in + q * rank_pitch_bytes,
 *           rank r's output at out + r * rank_pitch_bytes.  16-byte aligned, as is
 *           the pitch; the input rows and the output rows must not overlap.
 * count   : elements per rank; count * element size may not exceed
 *           SYMAR_STATIC_MAX_BYTES (else SYMAR_ERR_UNSUPPORTED -- use a heap).
 *           0 is a no-op.  The result is the same bits as allreduce() gives.
 * device_status : optional device word (may be NULL), owned by the caller; it is
 *           cleared on the stream before the launch and set to SYMAR_ERR_TIMEOUT
 *           if a bounded wait (0.2 s) inside the kernel gave up.  It is the ONLY report
 *           of a timeout: with NULL, a wait that gave up leaves `out` incomplete and
 *           nothing says so.  All CTAs of a call (at most 16 per rank) wait for one
 *           another and must be resident together: a GPU whose SMs are held by other
 *           kernels at that moment makes the waits run out.  SYMAR_ERR_UNSUPPORTED if
 *           the device could not hold the largest launch even when idle.
 * cuda_stream : the copy-free call enqueues one small memset (only if
 *           device_status is given) and one kernel.
 *
 * Set-up: the first call on each device looks up the device address of the
 * scratch array (with that device current) and loads the kernel; make that first
 * call outside any stream capture.  Sharing: all calls on a device use the same
 * array.  Its flags and counters are sequence numbers that are meant to persist
 * from call to call, so nothing needs clearing between calls, but two calls
 * that overlap on the GPU (different streams or host threads) race on it --
 * serialise them.                                                               */
enum { SYMAR_STATIC_MAX_BYTES = 32768 };
int allreduce_static(const void *in, void *out, size_t rank_pitch_bytes, int P, size_t count,
                     symar_dtype_t dtype, unsigned int *device_status, void *cuda_stream);

/* Test hook: one allreduce() of the given arguments through the instrumented kernel
 * instantiation, synchronously; *host_span_ns receives the time from the first CTA's start
 * (after its wait for the previous grid) to the last CTA's end on the device's nanosecond
 * timer (resolution about 32 ns): the protocol's own latency without the launch.  Not
 * capturable.  SYMAR_ERR_UNSUPPORTED for the bulk-copy kernel, which has no test hooks
 * (messages of 4 MiB per rank and more under SYMAR_TWOSHOT use the register kernel here).  */
int symar_debug_span(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype,
                     symar_algo_t algo, void *cuda_stream, double *host_span_ns);

/* Test hook: as symar_debug_span, with a stamp at every phase of the kernel.  Thread 0 of each
 * CTA stamps the device timer when it reaches phase k; host_ns (24 host doubles) receives, for
 * k = 0..7, {earliest, mean, latest} over all CTAs in nanoseconds since the earliest phase-0
 * stamp (-1 where the kernel has no such phase); host_stamps (8 host ints) the number of CTAs
 * that stamped phase k.  Phases: 0 = CTA in (after its wait for the previous grid); 7 = CTA out;
 * one-shot: 1 = every peer's signal seen, 2 = thread 0's loads back, reduced, store issued;
 * two-shot: 1 as one-shot, 2 = thread 0's share stored, 3 = the CTA's stores issued, 5 = release
 * fence done and "done" signal sent, 4 = every peer's "done" seen; LL: 1 = counter and input
 * back, stores issued, 3 = every peer's row seen, 4 = result stored.  Timer resolution ~32 ns.   */
int symar_debug_phases(symheap_t *heap, const void *in, void *out, size_t count, symar_dtype_t dtype,
                       symar_algo_t algo, void *cuda_stream, double *host_ns, int *host_stamps);

/* Self-test of the bounds-checking build of the library (libsymar_check.so, compiled with
 * -DSYMAR_CHECK: every heap address a kernel computes is checked against the region it must
 * lie in -- this call's input or output range, the LL, sentinel or atomic scratch, the flag
 * arrays, the counters -- and an access outside is recorded as SYMAR_ERR_INVAL in the status
 * word (rank, CTA slot, and in place of the peer the bit mask of the regions it was meant for:
 * 1 input, 2 output, 4 LL, 8 sentinel, 16 atomic scratch, 32 ready flags, 64 done flags,
 * 128 counters) and SKIPPED).  One CTA stores once inside a 64-byte output range and once
 * 64 bytes beyond it, at an address that is still inside the heap's user region (bytes 1024..1151
 * of rank 0; the heap needs 4 KiB per rank), so nothing can fault either way.  SYMAR_OK: the
 * first store landed, the second was recorded and kept out; SYMAR_ERR_UNSUPPORTED: this is
 * the regular build, which checks nothing.  Synchronous; clears the status word.          */
int symar_check_selftest(symheap_t *heap, void *cuda_stream);

/* Text of the last CUDA error seen by the library on this thread (host string). */
const char *symar_last_cuda_error(void);

/* ---- speed-of-light probes (Sec. VI: L_SoL = 2 L_L2_RTT + L_remote_store) ----
 *
 * Building blocks of the latency bound, measured on the box:
 * symar_probe_empty     enqueues an empty kernel of the given shape (its cost
 *                       in a stream or graph is the launch floor);
 * symar_probe_fence     ns per __threadfence() over a dependent chain with one
 *                       outstanding store each (the paper's L_L2_RTT estimate);
 * symar_probe_pingpong  ns per round trip of one 4-byte flag bounced between
 *                       two CTAs on different SMs through L2 (the one-GPU
 *                       analogue of the paper's two-GPU ping-pong); blocks 0
 *                       and 1 of a 2-block launch, usually neighbouring SMs.
 * The last two are synchronous and write host doubles.                         */
int symar_probe_empty(int grid_x, int grid_y, int block, void *cuda_stream);
/* the launch floor with programmatic dependent launch (see symar_set_pdl) */
int symar_probe_empty_pdl(int grid_x, int grid_y, int block, void *cuda_stream);
/* the same with the grid_y (2..8) CTAs of every column launched as one thread-block cluster, as
 * SYMAR_VARIANT_CLUSTER launches the ranks of a slot */
int symar_probe_empty_cluster(int grid_x, int grid_y, int block, void *cuda_stream);
int symar_probe_fence(int iterations, double *host_ns_per_fence);
int symar_probe_pingpong(int iterations, double *host_ns_per_round_trip);
/* The same between block 0 and block `partner_block` of a (partner_block + 1)-block
 * launch, i.e. between SMs that are farther apart the larger the partner index;
 * host_smids (2 ints, may be NULL) receives the two SM ids.  The round trip
 * depends on where the two SMs and the flag's L2 slice sit on the chip.        */
int symar_probe_pingpong_pair(int iterations, int partner_block, double *host_ns_per_round_trip,
                              int *host_smids);
/* The general form: a launch of `grid_blocks` one-thread blocks (2..1024) in which only
 * `first_block` (which sends first and takes the time) and `partner_block` play.  Measured
 * on B200: the round trip differs by up to 2x with the SM the FIRST block lands on and
 * hardly at all with the partner's, so a representative bound samples both.     */
int symar_probe_pingpong_blocks(int iterations, int first_block, int partner_block, int grid_blocks,
                                double *host_ns_per_round_trip, int *host_smids);

/* The barrier the method removes (Sec. III-B puts each such barrier above a microsecond): `ranks`
 * CTAs (2..32, one per rank, all co-resident) signal every peer and wait for every peer,
 * `iterations` times in a row; *host_ns_per_barrier is the mean as seen by rank 0.  ordered = 0:
 * relaxed signals and polls, as the paper measured; 1: release signals and acquire polls (a
 * barrier that also orders memory).  Synchronous; bounded spins (SYMAR_ERR_TIMEOUT).            */
int symar_probe_barrier(int ranks, int iterations, int ordered, double *host_ns_per_barrier);

/* ---- host side of the thread-level buffer primitives (symar_llbuffer.cuh; Sec. V
 *      "Host-side Functions": a scratch-size helper and the sentinel initialiser) ---- */

/* Bytes ONE rank's copy of an LLBuffer needs: sync_mode 0 = LL (every element occupies twice
 * its size), 1 = sentinel; elem_bytes 4 or 8; slots_per_cta elements per CTA and epoch; ctas
 * CTAs per rank; round_robin sub-buffers (0 counts as 1).  0 for bad arguments.              */
size_t symar_llbuffer_bytes(int sync_mode, size_t elem_bytes, size_t slots_per_cta, int ctas, int round_robin);

/* Fills `bytes` bytes of device memory with the sentinel (all ones) on the given stream:
 * what sentinel mode expects before the first send.  (LL mode expects zeros: cudaMemset.)   */
int symar_llbuffer_init_sentinel(void *device_ptr, size_t bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SYMAR_H */
