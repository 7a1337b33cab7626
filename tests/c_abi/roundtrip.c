/* The C ABI used from plain C: no Python, no torch.  Builds a small bf16-like cache on the host,
 * moves it through wm_checksum, wm_encode and wm_decode_verify on the device with buffers from
 * cudaMalloc, and checks the round trip, the checksums and that a flipped bit is refused.
 * Exit code 0 on success; prints one line. */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "wm.h"

#define CHECK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("cuda: %s\n", cudaGetErrorString(e_)); return 2; } } while (0)

static uint32_t lcg(uint32_t* s) { *s = *s * 1664525u + 1013904223u; return *s; }

int main(void)
{
    const uint64_t n = 37ull * 16384ull + 1234ull;
    const uint32_t chunk = 4u * 16384u;
    const uint64_t nc = wm_num_chunks(n, chunk), cap = wm_wire_bound(n, chunk), wsb = wm_workspace_bytes(n, chunk);
    uint8_t* host = (uint8_t*)malloc(n);
    uint32_t seed = 12345u;
    for (uint64_t i = 0; i + 1 < n; i += 2) {          /* exponents near 126, random sign and mantissa */
        uint32_t r = lcg(&seed);
        uint32_t v = ((r >> 31) << 15) | ((124u + ((r >> 8) & 3u) + ((r >> 10) & 1u)) << 7) | (r & 0x7Fu);
        host[i] = (uint8_t)v; host[i + 1] = (uint8_t)(v >> 8);
    }
    host[n - 1] = 0x5A;
    void *cache, *wire, *ws, *dst;
    uint32_t *crc_a, *crc_b, *crc_d;
    wm_result *res;
    CHECK(cudaMalloc(&cache, n)); CHECK(cudaMalloc(&wire, cap)); CHECK(cudaMalloc(&ws, wsb)); CHECK(cudaMalloc(&dst, n));
    CHECK(cudaMalloc((void**)&crc_a, 4 * nc)); CHECK(cudaMalloc((void**)&crc_b, 4 * nc)); CHECK(cudaMalloc((void**)&crc_d, 4 * nc));
    CHECK(cudaMalloc((void**)&res, sizeof(wm_result)));
    CHECK(cudaMemcpy(cache, host, n, cudaMemcpyHostToDevice));
    CHECK(cudaMemset(crc_d, 0, 4 * nc));
    cudaStream_t s;
    CHECK(cudaStreamCreate(&s));
    wm_result r_enc, r_dec, r_bad;
    for (int entropy = 0; entropy < 2; entropy++) {
        const uint32_t opt = entropy ? WM_OPT_ENTROPY : 0u;
        if (wm_checksum(cache, n, chunk, crc_a, ws, wsb, s) != WM_OK) { printf("wm_checksum refused\n"); return 1; }
        if (wm_encode_opt(cache, NULL, 0, n, chunk, NULL, crc_b, wire, cap, ws, wsb, opt, res, s) != WM_OK) { printf("wm_encode_opt refused\n"); return 1; }
        CHECK(cudaMemcpyAsync(&r_enc, res, sizeof r_enc, cudaMemcpyDeviceToHost, s));
        CHECK(cudaStreamSynchronize(s));
        if (r_enc.status != WM_OK || r_enc.wire_len >= n) { printf("encode: status %d wire_len %llu\n", r_enc.status, (unsigned long long)r_enc.wire_len); return 1; }
        if (wm_decode_verify_opt(wire, r_enc.wire_len, dst, NULL, 0, n, chunk, crc_d, ws, wsb, opt, res, s) != WM_OK) { printf("wm_decode_verify_opt refused\n"); return 1; }
        CHECK(cudaMemcpyAsync(&r_dec, res, sizeof r_dec, cudaMemcpyDeviceToHost, s));
        uint8_t* back = (uint8_t*)malloc(n);
        uint32_t* ca = (uint32_t*)malloc(4 * nc); uint32_t* cd = (uint32_t*)malloc(4 * nc);
        CHECK(cudaMemcpyAsync(back, dst, n, cudaMemcpyDeviceToHost, s));
        CHECK(cudaMemcpyAsync(ca, crc_a, 4 * nc, cudaMemcpyDeviceToHost, s));
        CHECK(cudaMemcpyAsync(cd, crc_d, 4 * nc, cudaMemcpyDeviceToHost, s));
        CHECK(cudaStreamSynchronize(s));
        if (r_dec.status != WM_OK || memcmp(back, host, n) != 0 || memcmp(ca, cd, 4 * nc) != 0 || r_dec.cache_crc != r_enc.cache_crc) {
            printf("round trip failed (entropy %d): status %d\n", entropy, r_dec.status); return 1;
        }
        /* one flipped payload bit: refused, the destination's checksums keep their values */
        uint8_t b;
        CHECK(cudaMemcpy(&b, (uint8_t*)wire + r_enc.wire_len - 9, 1, cudaMemcpyDeviceToHost));
        b ^= 0x20;
        CHECK(cudaMemcpy((uint8_t*)wire + r_enc.wire_len - 9, &b, 1, cudaMemcpyHostToDevice));
        if (wm_decode_verify_opt(wire, r_enc.wire_len, dst, NULL, 0, n, chunk, crc_d, ws, wsb, opt | WM_OPT_STRICT, res, s) != WM_OK) return 1;
        CHECK(cudaMemcpyAsync(&r_bad, res, sizeof r_bad, cudaMemcpyDeviceToHost, s));
        CHECK(cudaMemcpyAsync(cd, crc_d, 4 * nc, cudaMemcpyDeviceToHost, s));
        CHECK(cudaStreamSynchronize(s));
        if (r_bad.status == WM_OK || memcmp(ca, cd, 4 * nc) != 0) { printf("damaged image accepted (entropy %d)\n", entropy); return 1; }
        printf("entropy %d: ok, ratio %.4f, refused with status %d; ", entropy, (double)r_enc.wire_len / (double)n, r_bad.status);
        free(back); free(ca); free(cd);
    }
    printf("\n");
    return 0;
}
