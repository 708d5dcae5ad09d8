/*
 * aq_b200 -- AQ-SGD activation-delta codec for one NVIDIA B200 (sm_100a).
 *
 * C ABI of the boundary codec that AQ-SGD (Algorithm 1; two-machine form:
 * Algorithm 2 of the appendix "Distributed View") runs where one pipeline
 * stage hands its activations to the next:
 *
 *   sender    Delta_m = Q(a(xi) - m(xi));  m(xi) <- m(xi) + Delta_m;  send Delta_m
 *   receiver  m(xi) <- m(xi) + Delta_m;    use m(xi) as the forward activation
 *   backward  send Q(gradient) -- plain quantization, no buffer
 *
 * Q is the uniform b-bit quantizer of Section 4.1 ("Baselines"): a vector is
 * normalised into [-1,1] by its largest magnitude, [-1,1] is cut into 2^b equal
 * intervals and each number is sent as the b-bit number of its interval.  Here
 * a "vector" is a group of `group` consecutive hidden elements of one token:
 *
 *   s = max|d|,  Delta = s * 2^(1-b),  k = clamp(floor(d * (1/Delta)), -2^(b-1), 2^(b-1)-1),
 *   Q(d) = (k + 1/2) * Delta;   Delta < FLT_MIN  =>  Delta = 0, k = 0.
 *
 * All arithmetic is IEEE binary32, one rounding per operation (no fused
 * multiply-add), so results are reproducible bit for bit.
 *
 * One handle is ONE copy of the previous-message array m that Algorithm 1 sets
 * up, zero-filled, in its initialisation step: the sender's or the receiver's
 * side of one stage boundary.  A pipeline with K stages uses K-1 independent
 * pairs of handles (appendix A.1).
 *
 * Layouts (all row-major, densely packed):
 *   activations / gradients  T[n_batch][seq][hidden], T = fp16 or bf16 (2 bytes)
 *   m                        T[n_samples][seq][hidden], owned by the handle
 *   packed                   uint8[n_batch][seq*hidden*bits/8]; per sample a little-endian
 *                            bitstream: element j owns stream bits [j*bits, (j+1)*bits),
 *                            stream bit t is bit (t mod 8) of byte (t div 8); the field is
 *                            the two's-complement code k truncated to `bits` bits
 *   scales                   float[n_batch][seq][hidden/group], holds Delta of each group
 *
 * Pointers: unless a function says "host", every data pointer is a DEVICE
 * pointer (or any pointer the GPU can read, e.g. pinned host memory for
 * sample_ids), 16-byte aligned, owned by the caller, and must stay valid until
 * the work queued on the handle's stream has finished.  The functions only
 * enqueue work on that stream and return; they do not synchronise unless they
 * say so.  Calls on one handle must not overlap on the GPU (use one stream per
 * handle, or order the streams), and a handle is not thread-safe: one host thread at a
 * time.  Change AQ_STREAM only while the handle has no work in flight.
 *
 * Errors: functions returning int give AQ_OK or a negative AQ_E* code and leave
 * a message for aq_last_error().  Conditions only the GPU can see (a sample id
 * out of range, an id repeated inside one call, a first visit at the receiver
 * with no raw message) never fault: that sample is skipped -- no state change,
 * its outputs zero-filled -- and a sticky bit is set that aq_status() returns.
 * Preconditions that are not checked: finite inputs; both sides of a boundary
 * are fed the same sequence of sample ids.
 */
#ifndef AQ_B200_H
#define AQ_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aq_handle aq_handle;

enum {
  AQ_OK = 0,
  AQ_EINVAL = -1,        /* null / misaligned pointer, size or setting out of range */
  AQ_ENOMEM = -2,        /* device or host allocation failed */
  AQ_ECUDA = -3,         /* a CUDA runtime call failed; aq_last_error() names it */
  AQ_EUNSUPPORTED = -4   /* valid request that this build has no kernel for */
};

/* keys of aq_configure */
enum {
  AQ_DTYPE = 1,          /* AQ_FP16 (default) or AQ_BF16: type T of activations, gradients and m */
  AQ_BATCH = 2,          /* n_batch: sequences per aq_encode / aq_decode call, 0..4096 (default 1) */
  AQ_STREAM = 3,         /* cudaStream_t as an integer (default 0, the legacy default stream) */
  AQ_RAW = 4,            /* device pointer T[n_batch][seq][hidden]: the uncompressed message that
                            aq_decode stores for first-visit samples; 0 = none (default) */
  AQ_FIRST_FLAGS = 5,    /* device pointer uint8[n_batch] or 0: aq_encode / aq_decode write 1 for
                            each sample that took the first-visit path, else 0 */
  AQ_ROUNDING = 7,       /* AQ_ROUND_INTERVAL (default) or AQ_ROUND_STOCHASTIC: how aq_encode and
                            aq_quant_grad pick the code, see below */
  AQ_SEED = 8,           /* 64-bit key of the random numbers of AQ_ROUND_STOCHASTIC (default 0) */
  AQ_EPOCH = 9,          /* 64-bit counter that the caller sets before a call: two calls that should draw
                            independent random numbers need different values (for activations the epoch
                            or step number; for gradients any number unique to the call); default 0 */
  AQ_ROWS_PER_CTA = 6,   /* tuning: rows (256 chunks = 2048 elements each) that one CTA of aq_encode /
                            aq_decode walks; 0 (default) = chosen from the size of the call (1..4; on
                            large calls the CTAs that walk the last samples of aq_decode take half) */
  AQ_L2_PREFETCH = 10,   /* tuning: 1 (default for stores in device memory) = every CTA of aq_encode /
                            aq_decode asks for its rows of act and m, and every CTA of aq_quant_grad for its
                            piece of the gradient, to be brought into L2 ahead of its loads (bulk-prefetch
                            instructions, issued while the previous kernel of the stream drains; results
                            unchanged); act and grad must then be in device memory.  0 = plain loads only
                            (default for m of hosted stores, whose staged calls use the value set here) */
  AQ_RAW_LIST = 11       /* device pointer to an array of n_batch device pointers, or 0: the raw messages
                            of aq_decode_list, one per sample; a null entry = no raw message for that sample */
};
enum { AQ_FP16 = 0, AQ_BF16 = 1 };
/*
 * AQ_ROUND_INTERVAL: Q of Section 4.1 as described at the top of this file.
 * AQ_ROUND_STOCHASTIC: the unbiased Q that Theorem 3.1 assumes (its footnote sketches a randomised
 * rounding onto a uniform grid).  The 2^b levels reach from -s to +s,
 *   Delta = s / (2^(b-1) - 1/2),  k = clamp(floor(d * (1/Delta) + (r - 1/2))),  r uniform in [0,1),
 * so that E[(k + 1/2) * Delta] = d for every element of the group.  Receivers need no setting:
 * aq_decode / aq_dequant_grad rebuild (k + 1/2) * Delta from the Delta they are sent.  r comes
 * from Philox4x32-10 (Salmon et al., SC 2011), 16 bits per element: key = AQ_SEED, counter =
 * { chunk (element index / 8) inside the sample or gradient, sample id (0xFFFFFFFF for
 * gradients), AQ_EPOCH low word, AQ_EPOCH high word }; element j of a chunk takes bits
 * [16*(j%2), 16*(j%2)+16) of output word j/2 and r - 1/2 = (bits - 32767.5) * 2^-16.  The
 * result is a pure function of (seed, epoch, sample id, element, inputs).
 */
enum { AQ_ROUND_INTERVAL = 0, AQ_ROUND_STOCHASTIC = 1 };

/* sticky bits of aq_status */
enum {
  AQ_ST_BAD_ID = 1,      /* a sample id was < 0 or >= n_samples */
  AQ_ST_DUP_ID = 2,      /* an id appeared twice in one call; every occurrence after the first is skipped */
  AQ_ST_NO_RAW = 4,      /* aq_decode met a first-visit sample while AQ_RAW was 0 */
  AQ_ST_STAGED = 8,      /* a call after aq_prefetch brought another id at some position than the one
                            prefetched for it; that sample is skipped */
  AQ_ST_BAD_PTR = 16     /* a list-form call found a null or misaligned pointer in one of its arrays; nothing
                            is read or written for that sample */
};

/*
 * Initialisation step of Algorithm 1: allocates m (n_samples*seq*hidden*2 bytes of device
 * memory on the current device) filled with zeros, and an empty "seen before"
 * set.  bits in 1..8 is b of the forward quantizer; group (a multiple of 8, so that a group
 * is a whole number of 16-byte pieces and group*bits/8 whole bytes) must divide hidden, up to
 * group == hidden (one step per token).  The tuned kernels are those for groups of 8, 16, 32, 64, 128
 * and 256 elements -- the lanes that share a group's maximum are a power of two inside one warp;
 * any other multiple of 8 (24, 40, 48, 96, 320, 512 ...) runs on plainer kernels of its own: same
 * results by the same definition, at roughly 0.6 of the rate.  Those group sizes are offered by aq_create and
 * aq_create_hosted (every form of the calls, aq_quant_grad / aq_dequant_grad, either rounding mode);
 * the low-precision and binary32 stores answer AQ_EUNSUPPORTED for them.  Returns NULL on failure; aq_last_error(NULL) and aq_last_error_code(NULL)
 * say why.
 */
aq_handle* aq_create(int64_t n_samples, int seq, int hidden, int bits, int group);

/*
 * The same, with m in page-locked host memory instead of device memory (Section 3.3: the
 * previous messages can live in host memory; the appendix on offloading measures no loss of
 * throughput).  The GPU addresses that memory directly, so aq_encode / aq_decode and every other
 * call work unchanged and give the same results; they then run at the speed of the host link
 * (each element of m crosses it once in each direction) and the state is bounded by host
 * memory, not by the 180 GB of the GPU.  Run such a handle on its own stream beside the stage's
 * compute, as the paper hides the transfers behind the forward pass.
 */
aq_handle* aq_create_hosted(int64_t n_samples, int seq, int hidden, int bits, int group);

/*
 * Hosted handles only (AQ_EUNSUPPORTED otherwise): fetch m(xi) of the NEXT aq_encode / aq_decode
 * call ahead of time (Section 3.3 and the appendix on offloading: the previous messages are
 * prefetched from host memory while the preceding stages compute, so the transfer is off the
 * critical path).  sample_ids_host int32[n] (host; copied before the call returns), n must equal
 * AQ_BATCH now and at that call.  The call returns at once; on a stream of the handle's own
 * each sample's row of m is copied into a staging block in device memory (n rows, allocated at
 * the first use and when n grows): by one copy per row, or by one kernel when there are more than
 * 64 rows or rows under 64 KB.  Two staging blocks are used in turn and the rows travel home on a
 * second stream, so the fetch for call N+1 may be asked for as soon as call N is issued: it runs
 * beside call N's kernel and beside the write-back of call N's rows (both directions of the host
 * link at once) and waits only for what it must -- the write-back of the block it reuses, the
 * write-back of call N where both calls touch a sample, and calls that worked on the host block in
 * place.
 * The next aq_encode / aq_decode (aq_encode_host / aq_decode_host too) then
 *   - waits on the device, not on the host, until the rows have arrived,
 *   - runs the same kernel on the staged rows at device-memory speed, with the same results as
 *     on the host block in place, and
 *   - starts the copy of the rows back to host memory on the second stream, again without
 *     blocking the caller; every later call that touches m in place waits for it on the device.
 * That call must bring the prefetched ids, position by position: a sample whose id differs is
 * skipped (codes and scales zero, m untouched, as for a bad id) and AQ_ST_STAGED is set.  Ids
 * out of range and repeated ids are not fetched and the call reports them as always.  Between
 * aq_prefetch and the call that uses it, aq_import_sample of one of its samples is not seen by
 * that call.  A second aq_prefetch before the call replaces the first.  Calls with no prefetch
 * pending work on the host block in place.  Staged calls use events between two streams and
 * cannot be captured into a CUDA graph.
 */
int aq_prefetch(aq_handle* h, const int32_t* sample_ids_host, int n);

/*
 * The same, with the previous messages kept at low precision (appendix "Number of Bits for
 * Previous Messages": mz = z bits for m).  m is stored as m_bits-bit codes (2, 4 or 8) plus one
 * fp32 step per group of `group` elements -- Q of this file applied to m -- and takes
 * n_samples*seq*hidden*(m_bits/8 + 4/group) bytes.  Every visit works on the dequantized store:
 *   m_deq = (km + 1/2) * Delta_m;  sender: Delta = Q_b(act - m_deq);  m_new = m_deq + Delta (binary32);
 *   store <- Q_mbits(m_new);  the receiver's `out` is T(m_new);
 *   first visit: m_new = act (resp. the raw message), out = the raw message.
 * aq_encode / aq_decode and the host-buffer forms work as for aq_create.  AQ_ROUND_STOCHASTIC
 * applies to the message (Q_b) only: the store's own re-quantization always takes the interval
 * number, so that the receiver, which never learns the rounding mode, ends with the same store.
 * aq_state_checksum_noalloc answers AQ_EUNSUPPORTED on such a handle.  aq_state_checksum covers
 * the code bytes (as 32-bit words), then the steps, then the seen-set.  group must be 8, 16, 32, 64,
 * 128 or 256 (AQ_EUNSUPPORTED for the other multiples of 8).
 */
aq_handle* aq_create_lowbit(int64_t n_samples, int seq, int hidden, int bits, int group, int m_bits);

/*
 * The same, with the previous messages kept in binary32 (the precision of the paper's own runs:
 * 6.4 MB per 1024 x 1600 example): m_new = m + Delta is neither rounded to T nor re-quantized,
 * the receiver's `out` is T(m_new); 4 bytes per element of state.  Same restrictions as
 * aq_create_lowbit; aq_state_checksum covers the float words and the seen-set.
 */
aq_handle* aq_create_fp32(int64_t n_samples, int seq, int hidden, int bits, int group);

/*
 * Both at once: the store of aq_create_lowbit (m_bits 2, 4 or 8) kept in page-locked host
 * memory as for aq_create_hosted -- codes and steps alike.  An 8-bit store moves 1.06 instead of
 * 2 bytes per element over the host link in each direction.  The calls work on the host block
 * in place, or after aq_prefetch on staged rows (codes and steps).  (Not offered for the binary32 store: its
 * kernels read two 16-byte pieces 32 bytes apart per thread, which device memory serves at full
 * speed and the host link at a fifth of it.)
 */
aq_handle* aq_create_hosted_lowbit(int64_t n_samples, int seq, int hidden, int bits, int group, int m_bits);

/* Waits for the handle's stream, frees everything the handle owns.  NULL is allowed. */
void aq_destroy(aq_handle* h);

int aq_configure(aq_handle* h, int key, int64_t value);

/*
 * Sender side (Algorithm 2, the part run on network a; Algorithm 1, the test whether xi was seen before).  For each
 * of the n_batch samples, in one fused pass over the data:
 *   first visit  m(xi) <- act (bit copy; the full-precision activation itself is the
 *                message, the caller forwards `act`), codes and scales of the sample = 0;
 *   otherwise    d = act - m(xi); per group: Delta, codes k; m(xi) <- T(m(xi) + (k+1/2)*Delta).
 * act T[n_batch][seq][hidden] (in), sample_ids int32[n_batch] (in),
 * packed and scales (out, layouts above).
 */
int aq_encode(aq_handle* h, const void* act, const int32_t* sample_ids, void* packed, float* scales);

/*
 * Receiver side (Algorithm 2, the part run on network b): m(xi) <- T(m(xi) + (k+1/2)*Delta) on this
 * handle's own copy of m, and out <- the new m(xi), which network b uses as its forward
 * activation.  First visit: m(xi) <- raw, out <- raw (AQ_RAW).
 * packed, scales (in), sample_ids int32[n_batch] (in), out T[n_batch][seq][hidden] (out).
 */
int aq_decode(aq_handle* h, const void* packed, const float* scales, const int32_t* sample_ids, void* out);

/*
 * List forms of the two calls, for a stage that produces its micro-batches one at a time (GPipe-style
 * pipeline parallelism, Section 2: the micro-batches of a macro-batch cross the boundary one by one) and
 * wants several of them, each in a buffer of its own, to go through one launch: instead of one base
 * pointer per buffer the call takes DEVICE arrays of n_batch device pointers, entry y naming the buffer
 * of sample y -- act_list[y] T[seq][hidden], packed_list[y] uint8[seq*hidden*bits/8], scales_list[y]
 * float[seq*hidden/group], out_list[y] T[seq][hidden]; the raw messages of first visits come from
 * AQ_RAW_LIST.  Every pointer must be 16-byte aligned; the kernels check (the host cannot see the
 * arrays): a null or misaligned entry skips that sample altogether and sets AQ_ST_BAD_PTR.  Same
 * kernels, same results as the base-pointer forms on the same samples.  The arrays are read when the
 * kernel runs and must stay unchanged until then.  16-bit stores only (aq_create, aq_create_hosted);
 * AQ_EUNSUPPORTED otherwise.
 */
int aq_encode_list(aq_handle* h, const void* const* act_list, const int32_t* sample_ids,
                   void* const* packed_list, float* const* scales_list);
int aq_decode_list(aq_handle* h, const void* const* packed_list, const float* const* scales_list,
                   const int32_t* sample_ids, void* const* out_list);

/*
 * Backward direction (Algorithm 1, the message from machine b back to machine a: the quantized
 * gradient with respect to the activation): the same Q applied directly to the gradient; touches no state.  n_elems must be a
 * multiple of the handle's group; bits in 1..8 may differ from the handle's forward b.
 * grad T[n_elems] (in); packed uint8[n_elems*bits/8], scales float[n_elems/group] (out).
 * n_elems == 0 is a no-op.
 */
int aq_quant_grad(aq_handle* h, const void* grad, int64_t n_elems, int bits, void* packed, float* scales);

/* Inverse: out[j] = T((k_j + 1/2) * Delta).  packed, scales (in); out T[n_elems] (out). */
int aq_dequant_grad(aq_handle* h, const void* packed, const float* scales, int64_t n_elems, int bits, void* out);

/*
 * 64-bit digest of the whole state, independent of summation order:
 *   sum_i mix(i, word_i) + sum_xi mix(2^40 + xi, seen[xi])   (mod 2^64),
 * word_i = the i-th little-endian 64-bit word of m (four elements), mix(i, w) = the splitmix64 output
 * function applied to i*0x9E3779B97F4A7C15 + w.  Two handles fed the same id sequence
 * (the two sides of a boundary: in Algorithm 2 either network keeps its own copy of m)
 * must give the same digest.  Synchronises the stream; *out_host is host memory.
 */
int aq_state_checksum(aq_handle* h, uint64_t* out_host);

/*
 * The same digest as aq_state_checksum, for callers that cannot allocate device memory at the
 * time of the call: a process whose device memory was all handed out at start-up (a framework's
 * caching pool owns it and cudaMalloc would fail or evict), a step loop that must not take the
 * device-wide synchronisation that cudaMalloc / cudaFree can bring, a service with a fixed memory
 * budget per library.  (The paper has no counterpart; this entry point exists for such callers
 * only.)  Its working memory is a fixed array inside the library image -- 512 KiB of device
 * memory that every GPU which loads the library holds until the process exits -- so the call
 * itself runs no cudaMalloc, cudaFree or other allocating routine, and uses none of the handle's
 * own scratch.
 *   - Limit: m of at most 64 GiB (65536 slabs of 1 MiB, one partial sum each); a larger
 *     state is refused with AQ_EUNSUPPORTED and a message, nothing is launched.  16-bit stores
 *     only (aq_create, aq_create_hosted); AQ_EUNSUPPORTED for the low-precision and binary32 stores.
 *   - The first call on each device does the set-up: it looks up the array's device address
 *     (once per device, with that device current) and keeps it.  Make that first call before any
 *     stream capture begins.  A cudaDeviceReset invalidates the address that was kept; do not
 *     call again after one.
 *   - Every call, on any handle, uses the same array and leaves its partial sums there; each
 *     call rewrites every slot it reads, so nothing has to be cleared.  Calls that overlap
 *     on one GPU (different streams, different threads) race on the array and return
 *     garbage: keep them ordered.
 * Like aq_state_checksum it queues its kernels on the handle's stream, copies the 8-byte result
 * to the host and synchronises that stream before it returns; *out_host is host memory.
 */
int aq_state_checksum_noalloc(aq_handle* h, uint64_t* out_host);

/* Synchronises the stream, returns the sticky AQ_ST_* bits in *bits_host (host) and clears them. */
int aq_status(aq_handle* h, uint32_t* bits_host);

/* Message of the last failed call on this handle; with h == NULL, of the last failed
 * aq_create on this thread.  Never NULL.  The string is owned by the library. */
const char* aq_last_error(aq_handle* h);
/* The AQ_E* code that goes with that message (the aq_create family returns NULL, not a code):
 * AQ_EINVAL for arguments that no quantizer setting can have, AQ_EUNSUPPORTED for a valid setting
 * without a kernel, AQ_ENOMEM / AQ_ECUDA for the allocation. */
int aq_last_error_code(aq_handle* h);

/* Bytes of `packed` and floats of `scales` per sample for this handle's forward settings. */
int64_t aq_packed_bytes_per_sample(aq_handle* h);
int64_t aq_scales_per_sample(aq_handle* h);
/* Bytes of one sample's stored m, the size of the host buffer of aq_export_sample / aq_import_sample:
 * seq*hidden*2, or for a low-precision store the code bytes followed by the fp32 steps. */
int64_t aq_m_bytes_per_sample(aq_handle* h);

/*
 * Host-buffer forms: same operations, but every pointer is HOST memory (pinned memory
 * makes the copies asynchronous to the CPU; pageable works).  The call copies the inputs
 * to device staging buffers owned by the handle (allocated on first use, sized for the
 * current AQ_BATCH), runs the same kernel, copies the results back and returns when they
 * have arrived.  raw_host may be NULL (then first visits at the receiver are
 * skipped and reported, as with AQ_RAW = 0).  From 8 samples per call on, and when every id
 * is in range and appears once, the batch moves in four pieces: the copy in of one piece, the
 * kernel of the one before and the copy out of the one before that run together (two more
 * streams of the handle's own, ordered against the handle's stream by events); the results
 * do not depend on it.
 */
int aq_encode_host(aq_handle* h, const void* act_host, const int32_t* sample_ids_host,
                   void* packed_host, float* scales_host);
int aq_decode_host(aq_handle* h, const void* packed_host, const float* scales_host,
                   const void* raw_host, const int32_t* sample_ids_host, void* out_host);

/*
 * The wire between the two sides of a boundary when both live in one process: copies what
 * aq_encode produced for the handle's n_batch sequences -- the codes, the steps and, when
 * raw_src is given (a call with first visits; Algorithm 1: the first message of a sample is
 * the activation itself), the uncompressed block -- from the sender's device to buffers on
 * dst_device (the same device, or a peer over NVLink; plain copies into the receiver's own
 * memory, after which aq_decode reads locally).  Queued on the sender handle's stream `h`; the
 * receiver's stream has to wait for it (an event, or the same stream).  All pointers are device
 * pointers; *_dst live on dst_device.
 */
int aq_wire_copy(aq_handle* h, int dst_device, void* packed_dst, float* scales_dst, void* raw_dst,
                 const void* packed_src, const float* scales_src, const void* raw_src);

/*
 * The same wire in the backward direction (Algorithm 2: the receiving stage sends the quantized
 * gradient of the activation back to the sending stage): copies what aq_quant_grad produced for
 * n_elems elements at `bits` bits -- n_elems*bits/8 bytes of codes and n_elems/group steps -- to
 * buffers on dst_device, on the handle's stream.  Same rules as aq_wire_copy.  With both ends on
 * the handle's own device either call is a single kernel launch.
 */
int aq_wire_copy_grad(aq_handle* h, int dst_device, void* packed_dst, float* scales_dst,
                      const void* packed_src, const float* scales_src, int64_t n_elems, int bits);

/*
 * State access for checkpoints and tests.  Copies one sample's m block
 * (aq_m_bytes_per_sample bytes) and its seen flag between the handle and HOST memory;
 * synchronises the stream.
 */
int aq_export_sample(aq_handle* h, int64_t sample_id, void* m_host, uint8_t* seen_host);
int aq_import_sample(aq_handle* h, int64_t sample_id, const void* m_host, uint8_t seen);

#ifdef __cplusplus
}
#endif
#endif /* AQ_B200_H */
