/* pipeline_timing.c -- wall-clock timing of the pipelined transfers from plain C: only include/fastrack.h and the
 * CUDA runtime, no Python or torch on the timed path.  Built and run by bench.py; prints one JSON object per cell.
 *
 *   pipeline_timing h2d <len> <reps> <batches> <chunk>:<streams> [<chunk>:<streams> ...]
 *   pipeline_timing d2h <len> <reps> <batches> <chunk>:<streams> [...]
 *
 * h2d (paper Section 4.3, decryption pipeline): the ciphertext of a len-byte buffer sits in page-locked host memory;
 *   a cell times fastrack_pipelined_h2d (copy + decrypt + verify, blocking) against the raw transfer of the same
 *   bytes in the same process -- one cudaMemcpyAsync on a stream plus cudaStreamSynchronize -- and against the
 *   unpipelined sequence (that copy, then fastrack_decrypt_verify on the same stream, then synchronise).
 * d2h: the mirror, fastrack_pipelined_d2h against a raw device-to-host copy.
 * Every figure is the mean over `reps` back-to-back calls, taken `batches` times: the median batch is reported
 * with the fastest and the slowest.  Before timing, the cell is checked once: plaintext equal to what was
 * encrypted and every verdict 1 (h2d), or ciphertext that decrypts to the plaintext (d2h). */
#define _POSIX_C_SOURCE 199309L
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#include "fastrack.h"

#define CHECK_CUDA(call)                                                                      \
    do {                                                                                      \
        cudaError_t e_ = (call);                                                              \
        if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_)); return 2; } \
    } while (0)
#define CHECK_FR(call)                                                                        \
    do {                                                                                      \
        int rc_ = (call);                                                                     \
        if (rc_ != FASTRACK_OK) { fprintf(stderr, "%s: fastrack error %d\n", #call, rc_); return 3; } \
    } while (0)

static double now_us(void)
{
    struct timespec ts;
    clock_gettime(CLOCK_MONOTONIC, &ts);
    return (double)ts.tv_sec * 1e6 + (double)ts.tv_nsec * 1e-3;
}

static int cmp_double(const void* a, const void* b)
{
    const double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}

#define MAX_BATCHES 64
typedef struct { double median, min, max; } stat_t;

static stat_t summarize(double* v, int n)
{
    stat_t s;
    qsort(v, (size_t)n, sizeof(double), cmp_double);
    s.min = v[0];
    s.max = v[n - 1];
    s.median = (n & 1) ? v[n / 2] : 0.5 * (v[n / 2 - 1] + v[n / 2]);
    return s;
}

int main(int argc, char** argv)
{
    if (argc < 6) {
        fprintf(stderr, "usage: %s h2d|d2h <len> <reps> <batches> <chunk>:<streams> ...\n", argv[0]);
        return 1;
    }
    const int h2d = strcmp(argv[1], "h2d") == 0;
    const size_t len = (size_t)strtoull(argv[2], NULL, 10);
    const int reps = atoi(argv[3]);
    int batches = atoi(argv[4]);
    if (!h2d && strcmp(argv[1], "d2h") != 0) return 1;
    if (len == 0 || reps < 1 || batches < 1) return 1;
    if (batches > MAX_BATCHES) batches = MAX_BATCHES;

    uint8_t key[32], iv[12];
    for (int i = 0; i < 32; i++) key[i] = (uint8_t)(11 * i + 3);
    for (int i = 0; i < 12; i++) iv[i] = (uint8_t)(0x50 + i);

    uint8_t *h_plain = NULL, *h_cipher = NULL, *h_tags = NULL, *h_back = NULL;
    uint8_t *d_plain = NULL, *d_cipher = NULL, *d_out = NULL, *d_tags = NULL;
    uint32_t *d_ok = NULL, *h_ok = NULL;
    const size_t max_tags = 16 * (len / 16 + 1);
    CHECK_CUDA(cudaMallocHost((void**)&h_plain, len));
    CHECK_CUDA(cudaMallocHost((void**)&h_cipher, len));
    CHECK_CUDA(cudaMallocHost((void**)&h_back, len));
    CHECK_CUDA(cudaMalloc((void**)&d_plain, len));
    CHECK_CUDA(cudaMalloc((void**)&d_cipher, len));
    CHECK_CUDA(cudaMalloc((void**)&d_out, len));
    uint64_t s = 88172645463325252ull;                       /* xorshift64: the payload's value does not matter for timing */
    for (size_t i = 0; i + 8 <= len; i += 8) {
        s ^= s << 13; s ^= s >> 7; s ^= s << 17;
        memcpy(h_plain + i, &s, 8);
    }
    for (size_t i = len & ~(size_t)7; i < len; i++) h_plain[i] = (uint8_t)i;
    CHECK_CUDA(cudaMemcpy(d_plain, h_plain, len, cudaMemcpyHostToDevice));
    cudaStream_t st;
    CHECK_CUDA(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));

    for (int a = 5; a < argc; a++) {
        size_t chunk = 0;
        int streams = 0;
        if (sscanf(argv[a], "%zu:%d", &chunk, &streams) != 2 || chunk == 0 || streams < 1 || streams > 8) {
            fprintf(stderr, "bad cell %s\n", argv[a]);
            return 1;
        }
        fastrack_ctx* ctx = NULL;
        CHECK_FR(fastrack_ctx_create(key, chunk, &ctx));
        const size_t K = fastrack_num_chunks(ctx, len);
        if (16 * K > max_tags) return 1;
        CHECK_CUDA(cudaMallocHost((void**)&h_tags, 16 * K));
        CHECK_CUDA(cudaMallocHost((void**)&h_ok, 4 * K));
        CHECK_CUDA(cudaMalloc((void**)&d_tags, 16 * K));
        CHECK_CUDA(cudaMalloc((void**)&d_ok, 4 * K));
        double t_pipe[MAX_BATCHES], t_raw[MAX_BATCHES], t_seq[MAX_BATCHES];
        stat_t pipe, raw, seq;

        if (h2d) {
            /* the sender's side, on the GPU for speed: ciphertext and tags of the buffer, brought to the host */
            CHECK_FR(fastrack_encrypt_tag(ctx, iv, d_plain, len, d_cipher, d_tags, st));
            CHECK_CUDA(cudaMemcpyAsync(h_cipher, d_cipher, len, cudaMemcpyDeviceToHost, st));
            CHECK_CUDA(cudaMemcpyAsync(h_tags, d_tags, 16 * K, cudaMemcpyDeviceToHost, st));
            CHECK_CUDA(cudaStreamSynchronize(st));
            /* check once */
            CHECK_CUDA(cudaMemset(d_out, 0, len));
            CHECK_CUDA(cudaMemset(d_ok, 0, 4 * K));
            CHECK_FR(fastrack_pipelined_h2d(ctx, iv, h_cipher, len, h_tags, d_out, d_ok, streams));
            CHECK_CUDA(cudaMemcpy(h_back, d_out, len, cudaMemcpyDeviceToHost));
            CHECK_CUDA(cudaMemcpy(h_ok, d_ok, 4 * K, cudaMemcpyDeviceToHost));
            if (memcmp(h_back, h_plain, len) != 0) { fprintf(stderr, "plaintext mismatch\n"); return 4; }
            for (size_t k = 0; k < K; k++)
                if (h_ok[k] != 1u) { fprintf(stderr, "chunk %zu rejected\n", k); return 4; }
            for (int w = 0; w < 3; w++) CHECK_FR(fastrack_pipelined_h2d(ctx, iv, h_cipher, len, h_tags, d_out, d_ok, streams));
            for (int b = 0; b < batches; b++) {
                double t0 = now_us();
                for (int r = 0; r < reps; r++) CHECK_FR(fastrack_pipelined_h2d(ctx, iv, h_cipher, len, h_tags, d_out, d_ok, streams));
                t_pipe[b] = (now_us() - t0) / reps;
                t0 = now_us();
                for (int r = 0; r < reps; r++) {
                    CHECK_CUDA(cudaMemcpyAsync(d_out, h_cipher, len, cudaMemcpyHostToDevice, st));
                    CHECK_CUDA(cudaStreamSynchronize(st));
                }
                t_raw[b] = (now_us() - t0) / reps;
                t0 = now_us();
                for (int r = 0; r < reps; r++) {
                    CHECK_CUDA(cudaMemcpyAsync(d_cipher, h_cipher, len, cudaMemcpyHostToDevice, st));
                    CHECK_CUDA(cudaMemcpyAsync(d_tags, h_tags, 16 * K, cudaMemcpyHostToDevice, st));
                    CHECK_FR(fastrack_decrypt_verify(ctx, iv, d_cipher, len, d_tags, d_out, d_ok, st));
                    CHECK_CUDA(cudaStreamSynchronize(st));
                }
                t_seq[b] = (now_us() - t0) / reps;
            }
        } else {
            CHECK_FR(fastrack_pipelined_d2h(ctx, iv, d_plain, len, d_cipher, h_cipher, h_tags, streams));
            /* check once: the GPU decrypts and verifies what arrived on the host */
            CHECK_CUDA(cudaMemset(d_ok, 0, 4 * K));
            CHECK_FR(fastrack_pipelined_h2d(ctx, iv, h_cipher, len, h_tags, d_out, d_ok, streams));
            CHECK_CUDA(cudaMemcpy(h_back, d_out, len, cudaMemcpyDeviceToHost));
            CHECK_CUDA(cudaMemcpy(h_ok, d_ok, 4 * K, cudaMemcpyDeviceToHost));
            if (memcmp(h_back, h_plain, len) != 0) { fprintf(stderr, "round trip mismatch\n"); return 4; }
            for (size_t k = 0; k < K; k++)
                if (h_ok[k] != 1u) { fprintf(stderr, "chunk %zu rejected\n", k); return 4; }
            for (int w = 0; w < 2; w++) CHECK_FR(fastrack_pipelined_d2h(ctx, iv, d_plain, len, d_cipher, h_cipher, h_tags, streams));
            for (int b = 0; b < batches; b++) {
                double t0 = now_us();
                for (int r = 0; r < reps; r++) CHECK_FR(fastrack_pipelined_d2h(ctx, iv, d_plain, len, d_cipher, h_cipher, h_tags, streams));
                t_pipe[b] = (now_us() - t0) / reps;
                t0 = now_us();
                for (int r = 0; r < reps; r++) {
                    CHECK_CUDA(cudaMemcpyAsync(h_back, d_plain, len, cudaMemcpyDeviceToHost, st));
                    CHECK_CUDA(cudaStreamSynchronize(st));
                }
                t_raw[b] = (now_us() - t0) / reps;
                t0 = now_us();
                for (int r = 0; r < reps; r++) {
                    CHECK_FR(fastrack_encrypt_tag(ctx, iv, d_plain, len, d_cipher, d_tags, st));
                    CHECK_CUDA(cudaMemcpyAsync(h_cipher, d_cipher, len, cudaMemcpyDeviceToHost, st));
                    CHECK_CUDA(cudaMemcpyAsync(h_tags, d_tags, 16 * K, cudaMemcpyDeviceToHost, st));
                    CHECK_CUDA(cudaStreamSynchronize(st));
                }
                t_seq[b] = (now_us() - t0) / reps;
            }
        }
        pipe = summarize(t_pipe, batches);
        raw = summarize(t_raw, batches);
        seq = summarize(t_seq, batches);
        printf("{\"direction\": \"%s\", \"len\": %zu, \"chunk\": %zu, \"K\": %zu, \"streams\": %d, \"reps\": %d, \"batches\": %d, "
               "\"pipelined_us\": %.2f, \"pipelined_us_min\": %.2f, \"pipelined_us_max\": %.2f, "
               "\"raw_copy_us\": %.2f, \"raw_copy_us_min\": %.2f, \"raw_copy_us_max\": %.2f, "
               "\"copy_then_kernel_us\": %.2f, "
               "\"pipelined_gbs\": %.3f, \"raw_gbs\": %.3f, \"fraction_of_raw\": %.4f, \"launches\": %llu}\n",
               h2d ? "h2d" : "d2h", len, chunk, K, streams, reps, batches, pipe.median, pipe.min, pipe.max, raw.median, raw.min,
               raw.max, seq.median, (double)len / pipe.median * 1e-3, (double)len / raw.median * 1e-3, raw.median / pipe.median,
               (unsigned long long)fastrack_launch_count(ctx));
        fflush(stdout);
        fastrack_ctx_destroy(ctx);
        cudaFreeHost(h_tags); cudaFreeHost(h_ok); cudaFree(d_tags); cudaFree(d_ok);
        h_tags = NULL; h_ok = NULL; d_tags = NULL; d_ok = NULL;
    }
    cudaStreamDestroy(st);
    cudaFreeHost(h_plain); cudaFreeHost(h_cipher); cudaFreeHost(h_back);
    cudaFree(d_plain); cudaFree(d_cipher); cudaFree(d_out);
    return 0;
}
