/*
 * fastrack.h -- C ABI of the GPU side of Fastrack's CPU<->GPU secure channel on NVIDIA B200.
 *
 * The library implements the one data-parallel path of the paper "Fastrack: Fast IO for Secure ML
 * using GPU TEEs" (arXiv 2410.15240): authenticated decryption of a buffer that arrived over PCIe,
 * its mirror (encryption + tagging of a buffer that is about to leave the GPU), and the chunked
 * overlap of the PCIe copies with those kernels.
 *
 * Scheme (paper Section 2.3 "AES-GCM", Section 4.2 "Multi-chaining authentication"): AES-256 in
 * counter mode plus the GMAC tag over GF(2^128), i.e. AES-256-GCM with 96-bit IVs and 128-bit tags.
 * A buffer of `len` bytes is split into K = ceil(len / chunk_bytes) chunks; chunk k covers bytes
 * [k*chunk_bytes, min(len, (k+1)*chunk_bytes)), is an independent GCM message with empty AAD under
 *
 *     IV_k = iv_base[0..7] || BE32( (BE32(iv_base[8..11]) + k) mod 2^32 ),
 *
 * and has its own 16-byte tag at byte 16*k of the tag array.  Chunk order is bound by the index
 * inside IV_k: a chunk moved to another slot is decrypted under the wrong IV and rejected.
 * Within a chunk, keystream block j is E_K(IV_k || BE32(2 + j)); the tag is
 * GHASH_H(ciphertext zero-padded to 16 bytes || BE64(0) || BE64(8*len_k)) xor E_K(IV_k || BE32(1)).
 *
 * Conventions
 *   - Every function returns FASTRACK_OK (0) or a negative FASTRACK_ERR_* code.  Nothing throws,
 *     aborts or prints.  After FASTRACK_ERR_CUDA, fastrack_last_cuda_error(ctx) gives the CUDA code.
 *   - Pointers named d_* are DEVICE pointers on the context's device, 16-byte aligned.  Pointers named
 *     h_* are HOST pointers.  `key` and `iv_base` are always HOST pointers.  The caller owns every
 *     data buffer; the context owns only key-derived tables, per-chunk scratch and internal streams.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - A context is bound to the device that was current at creation.  That device must be the current device
 *     of the calling thread at every call that launches work or touches device memory; otherwise the call returns
 *     FASTRACK_ERR_ARG and does nothing.  A context must not be used from two host threads, or on two streams,
 *     at the same time (calls share scratch memory); the one exception is fastrack_verify, see there.
 *   - IV discipline is the caller's: one call consumes the IV values iv_base .. iv_base + K - 1;
 *     reusing an IV under the same key voids GCM's guarantees.  The library does not track this.
 *   - K is derived from `len`; dropping trailing chunks is invisible to this layer, so `len` must
 *     come from a trusted source.
 *   - There is no CPU implementation behind these calls: without a usable CUDA device they fail.
 *   - chunk_bytes may be anything from 16 bytes to 1 GiB.  Two kernel layouts serve that range -- a warp per run
 *     of 32 consecutive blocks of a chunk, or, when a launch has many chunks that are not large, a few lanes per
 *     chunk that take its blocks in turn -- and the library picks per launch; results do not depend on the choice.
 */
#ifndef FASTRACK_H
#define FASTRACK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define FASTRACK_API
#else
#define FASTRACK_API __attribute__((visibility("default")))
#endif

#define FASTRACK_OK               0
#define FASTRACK_ERR_ARG         -1   /* null pointer, misaligned or partially overlapping buffers, bad n_streams */
#define FASTRACK_ERR_CHUNK       -2   /* chunk_bytes is 0, not a multiple of 16, or above FASTRACK_MAX_CHUNK_BYTES */
#define FASTRACK_ERR_NOT_PINNED  -3   /* h_cipher_pinned is not page-locked host memory */
#define FASTRACK_ERR_CUDA        -4   /* a CUDA call failed; see fastrack_last_cuda_error */
#define FASTRACK_ERR_NOMEM       -5   /* host or device allocation failed */
#define FASTRACK_ERR_TOO_MANY    -6   /* more than 2^32 chunks in one call (the IV index is 32 bits) */
#define FASTRACK_ERR_LIMIT       -7   /* beyond a fixed limit of fastrack_decrypt_verify_noalloc (chunks per call, SMs of the device) */

/* Largest chunk: 1 GiB.  (GCM itself allows 2^36 - 32 bytes per message; the limit here keeps the
 * per-context table of powers of H, 16 bytes per 16-byte block of a chunk, at most 1 GiB.) */
#define FASTRACK_MAX_CHUNK_BYTES ((size_t)1 << 30)

/* Most chunks one fastrack_decrypt_verify_noalloc call may cover. */
#define FASTRACK_NOALLOC_MAX_CHUNKS 16384

typedef struct fastrack_ctx fastrack_ctx;

/* Context set-up (paper Section 2.3: one hash subkey H = E_K(0^128) serves the whole authentication;
 * Section 4.2: every chain uses the same H).
 * Copies the 32-byte AES-256 key (host pointer), expands it into the 15 round keys, derives H, and
 * builds on the current device the tables the kernels need, sized for `chunk_bytes`: the byte tables
 * of the fixed multiplier H^32 (and of H, for launches with many small chunks and for the sequential comparator) and the powers
 * H^0 .. H^(chunk_bytes/16 + 65), 16 bytes each, i.e. a table as large as one chunk.  Allocates device
 * memory and synchronises the device once.  chunk_bytes: multiple of 16, 16 .. FASTRACK_MAX_CHUNK_BYTES.
 * On success *out is a new context; on failure *out is NULL. */
FASTRACK_API int fastrack_ctx_create(const uint8_t key[32], size_t chunk_bytes, fastrack_ctx** out);

/* Zeroises the key material on host and device, frees tables, scratch and streams.  NULL is allowed.
 * Synchronises the device. */
FASTRACK_API void fastrack_ctx_destroy(fastrack_ctx* ctx);

/* K = ceil(len / chunk_bytes); 0 for len == 0 or ctx == NULL (Section 4.2: one tag per chunk). */
FASTRACK_API size_t fastrack_num_chunks(const fastrack_ctx* ctx, size_t len);

/* Kept for callers written against earlier versions, in which the scratch memory grew with the number of chunks
 * and this call pre-sized it.  The scratch is now a fixed set of records per context (the pieces of a chunk are
 * first combined inside a CTA, and only one record per CTA of a launch is needed across CTAs), allocated by
 * fastrack_ctx_create; no later call of any kind allocates device memory for it.  Returns FASTRACK_OK. */
FASTRACK_API int fastrack_ctx_reserve(fastrack_ctx* ctx, size_t max_len);

/* Paper-faithful framing (Section 4.2: one byte of additional authenticated data per chunk carries the chunk's
 * serial number; Section 4.4: that serial number defeats reordering).
 * chains_per_sample = n in 1..256: the buffer is a sequence of samples of n chunks each, and chunk k
 * authenticates the single byte (k mod n) as AAD (so the length block carries an AAD length of 8 bits).
 * chains_per_sample = 0 (the default at creation): AAD empty, chunk order bound by the IV index only.
 * The IV rule is unchanged in both cases.  Applies to every later call on the context, of every kind; both
 * ends must use the same setting (a mismatch rejects every chunk).  Takes effect for calls issued afterwards. */
FASTRACK_API int fastrack_ctx_set_framing(fastrack_ctx* ctx, unsigned chains_per_sample);

/* Test and tuning controls.  Results never depend on them -- every setting computes the same bytes, tags and
 * verdicts -- only the choice of kernel layout and launch geometry does, which the library otherwise makes by itself;
 * the defaults are the ones to ship.  They exist so that tests can force each layout on any shape and so that the
 * cost models can be re-fitted on new hardware.  The library reads no environment variable.
 * A setting applies to every later call on the context.  Unknown option: FASTRACK_ERR_ARG. */
enum {
    FASTRACK_OPT_ROW_SLOTS = 1,         /* row layout: spread a launch over this many warps (0 = automatic) */
    FASTRACK_OPT_GENERIC_SMEM = 2,      /* 1: portable shared-memory addressing even where the absolute form applies */
    FASTRACK_OPT_NO_OVERLAP_LAUNCH = 3, /* 1: plain stream-ordered launches (no programmatic dependent launch) */
    FASTRACK_OPT_STAGE_BYTES = 4,       /* pipelined calls: fixed stage size in bytes (0 = the shrinking / growing stages) */
    FASTRACK_OPT_DIRECT_SMALL = 5,      /* 0: single-stage pipelined transfers use the copy engine too (default 1) */
    FASTRACK_OPT_PACK_MAX_BLOCKS = 6,   /* packed layout only for chunks of at most this many blocks (0 = never; default and cap 4096) */
    FASTRACK_OPT_PACK_RUN = 7,          /* packed layout with this many counters per lane wherever it applies (0 = automatic) */
    FASTRACK_OPT_PACK_GROUP = 8,        /* packed layout: whole chunks per work item (0 = automatic) */
    FASTRACK_OPT_FOLD_TAIL = 9          /* row layout, fused passes: a chunk's last row of one or two blocks is worked on apart from
                                           its rows: 0 = where it pays (default), 1 = never, 2 = wherever a chunk ends that way;
                                           any other value: FASTRACK_ERR_ARG */
};
FASTRACK_API int fastrack_ctx_set_option(fastrack_ctx* ctx, int option, uint64_t value);

/* CUDA error code (cudaError_t as int) of the last failing CUDA call made through ctx, else 0. */
FASTRACK_API int fastrack_last_cuda_error(const fastrack_ctx* ctx);

/* GPU-side authenticated decryption (paper Section 4.2: the GPU decrypts and authenticates what it
 * received; decryption kernel = AES-CTR, authentication = GMAC per chunk; here one fused pass).
 *   iv_base  host, 12 bytes.
 *   d_cipher device, len bytes of ciphertext, chunks back to back.
 *   d_tags   device, 16*K bytes, tag of chunk k at byte 16*k.
 *   d_plain  device, len bytes out.  d_plain == d_cipher (exactly) is allowed: in-place.  Any other
 *            overlap with d_cipher is FASTRACK_ERR_ARG.
 *   d_ok     device, K uint32 out: 1 = all 128 tag bits match, 0 = rejected.
 * The plaintext of a rejected chunk is still written (Section 4.3 "eager evaluation" releases the
 * plaintext before the verdict; Section 3: results are discarded on failure) -- consult d_ok.
 * Asynchronous on `stream`: no host synchronisation; outputs are valid once the stream has been
 * synchronised.  len == 0 succeeds and writes nothing. */
FASTRACK_API int fastrack_decrypt_verify(fastrack_ctx* ctx, const uint8_t iv_base[12],
                                         const void* d_cipher, size_t len, const void* d_tags,
                                         void* d_plain, uint32_t* d_ok, void* stream);

/* GPU-side encryption with one tag per chunk, for GPU->CPU copies (paper Section 2.3: encryption is
 * the same keystream XOR; Section 4.2: one tag per chunk).
 *   d_plain  device, len bytes in.   d_cipher device, len bytes out (d_cipher == d_plain allowed).
 *   d_tags   device, 16*K bytes out.
 * Asynchronous on `stream`, same rules as fastrack_decrypt_verify. */
FASTRACK_API int fastrack_encrypt_tag(fastrack_ctx* ctx, const uint8_t iv_base[12],
                                      const void* d_plain, size_t len, void* d_cipher, void* d_tags,
                                      void* stream);

/* Pipelined host->device transfer with decryption and verification (paper Section 4.3 "Decryption
 * pipeline": the PCIe transfer is overlapped with the decryption and authentication kernels, so the
 * transfer costs max(copy, kernels) instead of their sum).
 * The buffer is cut into stages of whole chunks that shrink geometrically (three quarters of the buffer, then
 * three quarters of the rest, ... down to about 2 MiB, never less than one chunk); stage i is copied pinned->device into its
 * final place in d_plain with cudaMemcpyAsync on internal stream i mod n_streams and decrypted and verified
 * in place by the same kernels on that stream, so the copy of stage i+1 overlaps the kernels of stage i and
 * only the short last stage's kernel is exposed.
 *   h_cipher_pinned host, page-locked (cudaHostAlloc / cudaHostRegister), len bytes.
 *   h_tags          host, 16*K bytes, pinned or pageable (copied once, up front).
 *   d_plain, d_ok   device outputs as in fastrack_decrypt_verify.
 *   n_streams       1..8.
 * A transfer too small to be cut (one stage, up to about 3 MiB) is not copied at all: the kernel reads the
 * page-locked host buffer itself (and page-locked tags), which saves the copy engine's start-up latency.
 * BLOCKING: returns after every internal stream has completed, so wall-clock time around the call is
 * the effective transfer time.  Work already queued by the caller on other streams is not waited for. */
FASTRACK_API int fastrack_pipelined_h2d(fastrack_ctx* ctx, const uint8_t iv_base[12],
                                        const void* h_cipher_pinned, size_t len, const void* h_tags,
                                        void* d_plain, uint32_t* d_ok, int n_streams);

/* ---- A batch of samples, each with its own IV (paper Section 4.2) -------------------------------------------
 * The paper splits every input SAMPLE (an image, a sub-graph) into n chunks with n tags, and a batch holds many
 * samples that their owner encrypted one by one.  These two calls take such a batch in one launch:
 * n_samples samples of sample_bytes bytes each, back to back; sample s was (or is to be) encrypted as its own
 * multi-chain message under the 12-byte IV base d_iv_bases[12*s .. 12*s+11], i.e. its chunk k uses
 * IV = that base with k added to its last four bytes, and -- with fastrack_ctx_set_framing(ctx, n) -- the AAD
 * byte (k mod n).  A sample has ceil(sample_bytes / chunk_bytes) chunks, only its last may be short; tags and
 * verdicts are laid out sample after sample (sample s, chunk k at index s * chunks_per_sample + k).
 *   d_iv_bases   DEVICE, 12 * n_samples bytes (they normally arrive with the batch); no alignment needed.
 *   sample_bytes multiple of 16 (so that every sample stays 16-byte aligned).
 * The result is exactly what n_samples separate calls of fastrack_decrypt_verify / fastrack_encrypt_tag with
 * the respective IV bases would give, without their n_samples launches.  Asynchronous on `stream`; pointer and
 * overlap rules as for the single-buffer calls. */
FASTRACK_API int fastrack_decrypt_verify_samples(fastrack_ctx* ctx, const void* d_iv_bases, size_t sample_bytes,
                                                 size_t n_samples, const void* d_cipher, const void* d_tags,
                                                 void* d_plain, uint32_t* d_ok, void* stream);
FASTRACK_API int fastrack_encrypt_tag_samples(fastrack_ctx* ctx, const void* d_iv_bases, size_t sample_bytes,
                                              size_t n_samples, const void* d_plain, void* d_cipher, void* d_tags,
                                              void* stream);

/* fastrack_pipelined_h2d for such a batch (Sections 4.2 + 4.3 together): the batch sits in pinned host memory, its
 * IV bases (HOST pointer here, 12 * n_samples bytes, pinned or pageable) and tags travel with it; stages are whole
 * samples.  Blocking; everything else as in fastrack_pipelined_h2d and fastrack_decrypt_verify_samples. */
FASTRACK_API int fastrack_pipelined_h2d_samples(fastrack_ctx* ctx, const void* h_iv_bases, size_t sample_bytes,
                                                size_t n_samples, const void* h_cipher_pinned, const void* h_tags,
                                                void* d_plain, uint32_t* d_ok, int n_streams);

/* ---- Split passes (paper Section 4.3, "Eager evaluation") -------------------------------------------------
 * The paper lets the consumer start on the decrypted data before authentication has finished and runs the
 * authentication kernel later, in parallel with the next batch's PCIe transfer; results are discarded if the
 * verdict comes back negative (Section 3).  These two calls are the two halves of fastrack_decrypt_verify:
 *
 * fastrack_ctr_crypt: keystream + XOR only, d_out = d_in xor E_K(counter blocks).  It is its own inverse, so
 *   it both decrypts and encrypts.  No tags are read or written.  d_out == d_in is allowed.
 * fastrack_verify: GHASH of the CIPHERTEXT + tag compare only; d_cipher is not modified, d_ok as in
 *   fastrack_decrypt_verify.  The ciphertext must therefore still exist when it runs (do not decrypt in place
 *   if verification is deferred).  It uses a scratch bank of its own, so one fastrack_verify may run on
 *   another stream concurrently with one call of any other kind on the same context.
 * Both are asynchronous on `stream`; same pointer rules as fastrack_decrypt_verify.  For every input,
 * ctr_crypt followed (or preceded) by verify gives exactly the plaintext and verdicts of the fused call. */
FASTRACK_API int fastrack_ctr_crypt(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_in, size_t len,
                                    void* d_out, void* stream);
FASTRACK_API int fastrack_verify(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher, size_t len,
                                 const void* d_tags, uint32_t* d_ok, void* stream);

/* ---- Sequential-chain comparator (paper Section 4.2, the baseline authentication kernel) ------------------
 * Same inputs, outputs and verdicts as fastrack_verify, computed the way the paper's starting point does it:
 * every chunk's GMAC chain is walked block by block by ONE thread (Section 4.2: the baseline evaluates the m
 * block multiplications of a chain one after the other), so the only parallelism is across chunks and the time falls as 1/K when
 * a buffer is cut into K chunks (Section 5.3: 16 chains, up to 16x).  It exists to reproduce that curve next
 * to the parallel kernels; do not use it for throughput.  Asynchronous on `stream`; needs no scratch. */
FASTRACK_API int fastrack_verify_sequential(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher,
                                            size_t len, const void* d_tags, uint32_t* d_ok, void* stream);

/* ---- Keystream ahead of the data (paper Section 4.3, "Parallel AES evaluation") --------------------------
 * AES(k, counter) does not depend on the ciphertext, so the one-time pad can be produced while the PCIe copy
 * is still in flight; when the data arrives, decryption is one XOR.
 *
 * fastrack_keystream: writes the keystream of a len-byte buffer to d_pad (device, len bytes, same chunk
 *   layout as the data) and E_K(IV_k || 1), the tag mask of every chunk, to d_mask (device, 16*K bytes).
 * fastrack_xor_verify: d_plain = d_cipher xor d_pad, GHASH of the ciphertext, tag = GHASH xor d_mask[k],
 *   compare -> d_ok.  No AES runs in this pass.  d_plain == d_cipher is allowed; d_pad must not overlap d_plain.
 *   d_pad / d_mask must come from fastrack_keystream with the same context, iv_base and len.
 * fastrack_pipelined_h2d_ahead: fastrack_pipelined_h2d with the keystream of the whole buffer produced first,
 *   on an internal stream, under the first copy; the per-stage kernels then only XOR and authenticate, which
 *   shortens the one kernel no copy hides (the last stage's).  d_pad: caller-provided device buffer of len
 *   bytes, 16-byte aligned, not overlapping d_plain; its contents afterwards are the keystream (treat it as
 *   secret and clear it).  Blocking, like fastrack_pipelined_h2d. */
FASTRACK_API int fastrack_keystream(fastrack_ctx* ctx, const uint8_t iv_base[12], size_t len, void* d_pad,
                                    void* d_mask, void* stream);
FASTRACK_API int fastrack_xor_verify(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher, size_t len,
                                     const void* d_pad, const void* d_mask, const void* d_tags, void* d_plain,
                                     uint32_t* d_ok, void* stream);
FASTRACK_API int fastrack_pipelined_h2d_ahead(fastrack_ctx* ctx, const uint8_t iv_base[12],
                                              const void* h_cipher_pinned, size_t len, const void* h_tags,
                                              void* d_pad, void* d_plain, uint32_t* d_ok, int n_streams);

/* fastrack_decrypt_verify for callers that must not allocate.  (The paper has no counterpart; this is a
 * deployment variant of the same operation.)
 * Who needs it: code that runs after start-up in a process whose device memory is fully owned by another
 * allocator or a fixed budget, or inside a serving loop where the device-wide synchronisation that comes with
 * a device allocation would stall every other stream.  The guarantee is part of this call's contract: it calls
 * no cudaMalloc, cudaFree or other allocating routine, and the records in which the CTAs of a launch combine
 * their pieces of a chunk are a fixed array inside the library image (32 KiB, held by every GPU that loads the
 * library until the process exits) rather than memory of the context.  (fastrack_decrypt_verify keeps its
 * records in the context; they have a fixed size and are allocated by fastrack_ctx_create, but that call's
 * contract does not promise it.)
 * Arguments, outputs, alignment and overlap rules, and asynchrony on `stream` are exactly those of
 * fastrack_decrypt_verify, and the results are bit-identical to it.  Differences:
 *   - at most FASTRACK_NOALLOC_MAX_CHUNKS chunks per call; more returns FASTRACK_ERR_LIMIT and does nothing;
 *   - the context's device must be the current device (else FASTRACK_ERR_ARG);
 *   - the first call on each device looks up the array's device address (cudaGetSymbolAddress); make that
 *     first call during start-up, before any stream capture begins;
 *   - all calls on a device share the one array, which still holds what the previous call left: each call
 *     first zeroes the part it will use, on `stream`.  Two calls whose GPU work overlaps (different streams,
 *     different contexts or different host threads) race on it and produce wrong verdicts -- keep every
 *     call of this entry point on one stream, or order them with events. */
FASTRACK_API int fastrack_decrypt_verify_noalloc(fastrack_ctx* ctx, const uint8_t iv_base[12],
                                                 const void* d_cipher, size_t len, const void* d_tags,
                                                 void* d_plain, uint32_t* d_ok, void* stream);

/* Pipelined device->host transfer with encryption and tagging: the mirror of fastrack_pipelined_h2d for
 * GPU->CPU copies (paper Section 2.3: encryption is the same keystream XOR; Section 4.2: one tag per chunk;
 * Section 4.3: the transfer is overlapped with the kernels).
 * The buffer is cut into stages of whole chunks that GROW geometrically (about 2 MiB first, then four times as much,
 * ... the last one about three quarters of the buffer); stage i is encrypted and tagged from d_plain into d_cipher on
 * internal stream i mod n_streams and then copied, with its tags, to the host on the same stream, so the copy
 * of stage i overlaps the kernel of stage i+1 and only the short first stage's kernel is exposed.
 *   d_plain         device, len bytes in (not modified unless d_cipher == d_plain).
 *   d_cipher        device, len bytes of ciphertext staging; d_cipher == d_plain (exactly) encrypts in place.
 *                   Otherwise its contents after the call are unspecified: a transfer too small to be cut (one
 *                   stage, up to about 3 MiB) is written to the host buffers by the kernel itself and skips it.
 *   h_cipher_pinned host, page-locked, len bytes out.
 *   h_tags          host, 16*K bytes out, pinned or pageable.  Page-locked is the fast form: the tags of a stage then
 *                   leave with that stage; tags bound for pageable memory are copied once, after the last stage
 *                   (a device-to-host copy into pageable memory blocks the host, which would stall the pipeline).
 *   n_streams       1..8.
 * BLOCKING: returns when the ciphertext and the tags are complete in host memory. */
FASTRACK_API int fastrack_pipelined_d2h(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_plain, size_t len,
                                        void* d_cipher, void* h_cipher_pinned, void* h_tags, int n_streams);

/* fastrack_pipelined_d2h for a batch of samples, each encrypted as its own multi-chain message under its own IV base
 * (Sections 4.2 + 4.3, outbound): n_samples samples of sample_bytes bytes (a multiple of 16) back to back in d_plain;
 * h_iv_bases is a HOST pointer to 12 * n_samples bytes (pinned or pageable; copied in once, up front); tags leave in
 * the order of fastrack_encrypt_tag_samples.  Stages are whole samples.  Blocking; everything else as in
 * fastrack_pipelined_d2h. */
FASTRACK_API int fastrack_pipelined_d2h_samples(fastrack_ctx* ctx, const void* h_iv_bases, size_t sample_bytes,
                                                size_t n_samples, const void* d_plain, void* d_cipher,
                                                void* h_cipher_pinned, void* h_tags, int n_streams);

/* Stage-level trace of pipelined host->device calls (paper Section 4.3 argues that the copy of one piece hides
 * the kernels of the previous one; this shows it).  While enabled, every fastrack_pipelined_h2d /
 * fastrack_pipelined_h2d_ahead call records three CUDA events per stage on the stage's stream -- before its copy,
 * after its copy, after its kernel -- and fastrack_ctx_get_trace returns, for the most recent call, each stage's
 * byte range, stream index and those three times in milliseconds since the first copy was started.
 * (A transfer small enough for the kernel to read the host buffer itself shows as one stage with an empty copy
 * interval.)  Enabling creates the events (allocation; do it at start-up); tracing adds about a microsecond per event.
 * fastrack_ctx_get_trace copies at most `cap` entries to `out` (may be NULL) and returns the number of stages. */
typedef struct {
    size_t offset, bytes;          /* byte range of the stage inside the buffer */
    int stream;                    /* index of the internal stream it ran on */
    float copy_start_ms, copy_end_ms, kernel_end_ms;
} fastrack_stage_trace;
FASTRACK_API int fastrack_ctx_set_trace(fastrack_ctx* ctx, int enable);
FASTRACK_API size_t fastrack_ctx_get_trace(const fastrack_ctx* ctx, fastrack_stage_trace* out, size_t cap);

/* Number of kernels the library launched through ctx since creation (data-path launches only;
 * cudaMemcpyAsync calls are not counted).  For benchmarks' bookkeeping. */
FASTRACK_API uint64_t fastrack_launch_count(const fastrack_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FASTRACK_H */
