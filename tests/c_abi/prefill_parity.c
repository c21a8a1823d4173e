/* Parity without Python in the loop: a C program that drives the CUDA library through its C ABI
 * (device memory from the CUDA runtime) and checks the result against the float64 CPU oracle
 * (oracle/lagkv_oracle.c, linked in).  Inputs: a counter-based hash turned into bf16 values with
 * per-channel scales, so that the channel ranges differ as they do in a real K cache.
 * Exit code 0 and "ok ..." on success. */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "lagkv.h"

int64_t lagkv_oracle_compress(const uint16_t *K, const uint16_t *V, int64_t B, int64_t H, int64_t seq_len, int64_t D,
                              int64_t static_len, int64_t L, int64_t k, int ddof, int variant, int storage,
                              int32_t *idx_out, uint16_t *K_out, uint16_t *V_out, double *scores_out);

static uint32_t mix(uint32_t x)
{
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}
/* roughly normal value (sum of four uniforms) times a per-channel scale, rounded to bf16 by truncation */
static uint16_t synth_bf16(uint32_t i, uint32_t channel, uint32_t seed)
{
    uint32_t h = mix(i * 2654435761u + seed);
    float u = 0.0f, scale, f;
    uint32_t bits;
    int j;
    for (j = 0; j < 4; ++j) { u += (float)(h & 0xffffu) / 65536.0f - 0.5f; h = mix(h + 0x9e3779b9u); }
    scale = 0.25f + (float)(mix(channel + 77u * seed) & 1023u) / 128.0f;
    f = u * 1.7f * scale;
    memcpy(&bits, &f, sizeof bits);
    return (uint16_t)(bits >> 16);
}

#define CHECK(cond, what) do { if (!(cond)) { fprintf(stderr, "prefill_parity: %s\n", what); return 1; } } while (0)

int main(void)
{
    const int B = 3, H = 2, D = 128, sink = 8, L = 256, k = 64, S = 8 + 6 * 256 + 100;
    const size_t n_in = (size_t)B * H * S * D;
    lagkv_config cfg;
    lagkv_plan_t plan = NULL;
    int64_t L_R, n_c = (S - sink) / L - 1;
    uint16_t *K = malloc(n_in * 2), *V = malloc(n_in * 2);
    uint16_t *Ko, *Vo, *Kr, *Vr;
    int32_t *idx, *idx_r, status[4];
    float *scores;
    double *scores_r, max_err = 0.0;
    void *dK, *dV, *dKo, *dVo, *dIdx, *dSc, *dWs;
    size_t ws_bytes, n_out, i;
    int mismatched = 0;

    for (i = 0; i < n_in; ++i) {
        K[i] = synth_bf16((uint32_t)i, (uint32_t)(i % D) + 1000u * (uint32_t)((i / ((size_t)S * D)) % H), 1u);
        V[i] = synth_bf16((uint32_t)i, (uint32_t)(i / D) % 97u, 2u);
    }
    memset(&cfg, 0, sizeof cfg);
    cfg.B = B; cfg.H_kv = H; cfg.D = D; cfg.sink = sink; cfg.lag = L; cfg.keep_k = k; cfg.keep_ratio = 0.25;
    cfg.std_ddof = 1; cfg.device = 0;
    CHECK(lagkv_plan(&cfg, &plan) == LAGKV_OK, "lagkv_plan");
    L_R = lagkv_compressed_len(plan, S, -1);
    CHECK(L_R == sink + k * n_c + L + (S - sink) % L, "Eq. 12");
    n_out = (size_t)B * H * L_R * D;
    ws_bytes = lagkv_workspace_bytes(plan, 0);
    CHECK(cudaMalloc(&dK, n_in * 2) == cudaSuccess && cudaMalloc(&dV, n_in * 2) == cudaSuccess &&
          cudaMalloc(&dKo, n_out * 2) == cudaSuccess && cudaMalloc(&dVo, n_out * 2) == cudaSuccess &&
          cudaMalloc(&dIdx, (size_t)B * H * L_R * 4) == cudaSuccess &&
          cudaMalloc(&dSc, (size_t)B * H * n_c * L * 4) == cudaSuccess && cudaMalloc(&dWs, ws_bytes) == cudaSuccess,
          "cudaMalloc");
    cudaMemcpy(dK, K, n_in * 2, cudaMemcpyHostToDevice);
    cudaMemcpy(dV, V, n_in * 2, cudaMemcpyHostToDevice);
    CHECK(lagkv_workspace_init(plan, dWs, ws_bytes, NULL) == LAGKV_OK, "workspace init");
    CHECK(lagkv_compress_prefill(plan, dK, dV, S, dKo, dVo, (int32_t *)dIdx, (float *)dSc, dWs, ws_bytes, NULL) == LAGKV_OK,
          "lagkv_compress_prefill");
    CHECK(lagkv_read_status(plan, dWs, NULL, status) == LAGKV_OK && status[0] == 0, "device status");

    Ko = malloc(n_out * 2); Vo = malloc(n_out * 2); Kr = malloc(n_out * 2); Vr = malloc(n_out * 2);
    idx = malloc((size_t)B * H * L_R * 4); idx_r = malloc((size_t)B * H * L_R * 4);
    scores = malloc((size_t)B * H * n_c * L * 4); scores_r = malloc((size_t)B * H * n_c * L * 8);
    cudaMemcpy(Ko, dKo, n_out * 2, cudaMemcpyDeviceToHost);
    cudaMemcpy(Vo, dVo, n_out * 2, cudaMemcpyDeviceToHost);
    cudaMemcpy(idx, dIdx, (size_t)B * H * L_R * 4, cudaMemcpyDeviceToHost);
    cudaMemcpy(scores, dSc, (size_t)B * H * n_c * L * 4, cudaMemcpyDeviceToHost);
    CHECK(lagkv_oracle_compress(K, V, B, H, S, D, sink, L, k, 1, 0, 0, idx_r, Kr, Vr, scores_r) == L_R, "oracle length");

    for (i = 0; i < (size_t)B * H * n_c * L; ++i) {
        double e = fabs((double)scores[i] - scores_r[i]);
        if (e > max_err) max_err = e;
    }
    CHECK(max_err <= 1e-4, "score error above 1e-4");
    CHECK(max_err * L / 2.0 <= 2e-5, "score error above 2e-5 of the mean score");
    for (i = 0; i < (size_t)B * H * L_R; ++i) mismatched += idx[i] != idx_r[i];
    CHECK(mismatched == 0, "kept indices differ from the oracle");
    CHECK(memcmp(Ko, Kr, n_out * 2) == 0 && memcmp(Vo, Vr, n_out * 2) == 0, "compacted rows differ from the oracle");
    lagkv_plan_destroy(plan);
    printf("ok L_R=%lld max_score_err=%.3e\n", (long long)L_R, max_err);
    return 0;
}
