/* roundtrip.c -- the library used from plain C: no Python, no torch, only the CUDA runtime for device memory.
 * Encrypts a buffer on the GPU, copies ciphertext and tags to the host and back through the pipelined call,
 * checks the plaintext and the verdicts, flips one ciphertext bit and one tag bit and checks that exactly those
 * two chunks are rejected.  Exit code 0 and a line "ok ..." on success.  Built and run by tests/test_c_abi.py. */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

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

int main(int argc, char** argv)
{
    const size_t chunk = argc > 1 ? (size_t)strtoull(argv[1], NULL, 10) : 65536;
    const size_t len = argc > 2 ? (size_t)strtoull(argv[2], NULL, 10) : (3u << 20) + 4099;
    uint8_t key[32], iv[12];
    for (int i = 0; i < 32; i++) key[i] = (uint8_t)(7 * i + 1);
    for (int i = 0; i < 12; i++) iv[i] = (uint8_t)(0xA0 + i);

    fastrack_ctx* ctx = NULL;
    CHECK_FR(fastrack_ctx_create(key, chunk, &ctx));
    const size_t K = fastrack_num_chunks(ctx, len);

    uint8_t *h_plain = NULL, *h_cipher = NULL, *h_tags = NULL, *h_back = (uint8_t*)malloc(len);
    uint32_t* h_ok = (uint32_t*)malloc(4 * K);
    CHECK_CUDA(cudaMallocHost((void**)&h_plain, len));
    CHECK_CUDA(cudaMallocHost((void**)&h_cipher, len));
    CHECK_CUDA(cudaMallocHost((void**)&h_tags, 16 * K));
    uint32_t s = 12345u;
    for (size_t i = 0; i < len; i++) { s = s * 1664525u + 1013904223u; h_plain[i] = (uint8_t)(s >> 24); }

    uint8_t *d_plain = NULL, *d_cipher = NULL, *d_tags = NULL, *d_out = NULL;
    uint32_t* d_ok = NULL;
    CHECK_CUDA(cudaMalloc((void**)&d_plain, len));
    CHECK_CUDA(cudaMalloc((void**)&d_cipher, len));
    CHECK_CUDA(cudaMalloc((void**)&d_out, len));
    CHECK_CUDA(cudaMalloc((void**)&d_tags, 16 * K));
    CHECK_CUDA(cudaMalloc((void**)&d_ok, 4 * K));
    CHECK_CUDA(cudaMemcpy(d_plain, h_plain, len, cudaMemcpyHostToDevice));

    /* GPU -> host: encrypt + tag with the copies overlapped */
    CHECK_FR(fastrack_pipelined_d2h(ctx, iv, d_plain, len, d_cipher, h_cipher, h_tags, 2));
    if (memcmp(h_cipher, h_plain, len < 64 ? len : 64) == 0) { fprintf(stderr, "ciphertext equals plaintext\n"); return 4; }

    /* tamper: one ciphertext bit in chunk 1, one tag bit in the last chunk */
    const size_t bad_a = K > 1 ? 1 : 0, bad_b = K - 1;
    h_cipher[bad_a * chunk + 5] ^= 0x08;
    h_tags[16 * bad_b + 9] ^= 0x80;

    /* host -> GPU: copy, decrypt and verify, pipelined */
    CHECK_FR(fastrack_pipelined_h2d(ctx, iv, h_cipher, len, h_tags, d_out, d_ok, 3));
    CHECK_CUDA(cudaMemcpy(h_back, d_out, len, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(h_ok, d_ok, 4 * K, cudaMemcpyDeviceToHost));
    size_t rejected = 0, wrong_bytes = 0;
    for (size_t k = 0; k < K; k++) {
        const int expect = !(k == bad_a || k == bad_b);
        if ((int)h_ok[k] != expect) { fprintf(stderr, "chunk %zu: verdict %u, expected %d\n", k, h_ok[k], expect); return 5; }
        rejected += !h_ok[k];
    }
    for (size_t i = 0; i < len; i++) wrong_bytes += h_back[i] != h_plain[i];
    if (wrong_bytes != 1 || h_back[bad_a * chunk + 5] == h_plain[bad_a * chunk + 5]) {
        fprintf(stderr, "%zu plaintext bytes differ, expected exactly the tampered one\n", wrong_bytes);
        return 6;
    }

    /* the device-resident calls on a caller's stream */
    cudaStream_t stream;
    CHECK_CUDA(cudaStreamCreate(&stream));
    CHECK_FR(fastrack_encrypt_tag(ctx, iv, d_plain, len, d_cipher, d_tags, stream));
    CHECK_FR(fastrack_decrypt_verify(ctx, iv, d_cipher, len, d_tags, d_cipher, d_ok, stream));      /* in place */
    CHECK_CUDA(cudaStreamSynchronize(stream));
    CHECK_CUDA(cudaMemcpy(h_back, d_cipher, len, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(h_ok, d_ok, 4 * K, cudaMemcpyDeviceToHost));
    for (size_t k = 0; k < K; k++)
        if (h_ok[k] != 1u) { fprintf(stderr, "round trip: chunk %zu rejected\n", k); return 7; }
    if (memcmp(h_back, h_plain, len) != 0) { fprintf(stderr, "round trip: plaintext differs\n"); return 8; }

    printf("ok len=%zu chunk=%zu K=%zu rejected=%zu launches=%llu\n", len, chunk, K, rejected,
           (unsigned long long)fastrack_launch_count(ctx));
    fastrack_ctx_destroy(ctx);
    cudaStreamDestroy(stream);
    cudaFree(d_plain); cudaFree(d_cipher); cudaFree(d_out); cudaFree(d_tags); cudaFree(d_ok);
    cudaFreeHost(h_plain); cudaFreeHost(h_cipher); cudaFreeHost(h_tags);
    free(h_back); free(h_ok);
    return 0;
}
