/* A plain C program that drives the library on a GPU with nothing but speca.h and the CUDA runtime:
 * no Python, no torch. It builds a small fp32 cache, feeds it features from a 32-bit linear
 * congruential generator over three reference steps (one of them masked), runs a forecast, the
 * verification and the continuation rule, and writes every result to a binary file that the test
 * harness compares with the CPU oracle on the same generated inputs.
 *
 * File layout (little endian): int32 header {B, n_entries, m, basis, n_steps}, then per entry
 * int32 {tokens, dim}; float fresh[B][N_v*D] (the verification feature that was used); then float
 * forecast[e][B][N_e*D] for every entry; float err[B]; uint8 accept[B]; uint8 next_active[B]; int32
 * spec_count[B]; int32 n_active.
 *
 * usage: gpu_roundtrip <out-file> <basis> [fused]
 * With a third argument the last reference step and the forecast are ONE call
 * (speca_cache_update_forecast) instead of speca_cache_update + speca_cache_commit_step + speca_forecast;
 * the file must come out the same.
 */
#include <speca.h>

#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#define B 3
#define NE 3
#define M 2

static const speca_entry_desc_t kEntries[NE] = {{7, 33}, {64, 257}, {19, 1031}};
static const double kTimes[3][B] = {{1.00, 0.99, 1.01}, {0.93, 0.92, 0.95}, {0.90, 0.0, 0.91}};
static const uint8_t kMask2[B] = {1, 0, 1}; /* third reference step: sample 1 sits out */
static const double kTarget[B] = {0.86, 0.88, 0.87};

#define CK(x)                                                            \
    do {                                                                 \
        if (!(x)) {                                                      \
            fprintf(stderr, "FAILED line %d: %s\n", __LINE__, #x);       \
            return 1;                                                    \
        }                                                                \
    } while (0)

/* Numerical Recipes' 32-bit generator; value = top 24 bits mapped to [-1, 1). */
static uint32_t g_state;
static float next_value(void) {
    g_state = g_state * 1664525u + 1013904223u;
    return (float)(g_state >> 8) * (1.0f / 8388608.0f) - 1.0f;
}

int main(int argc, char** argv) {
    speca_cache_config_t cfg;
    speca_cache_t* cache = NULL;
    size_t bytes = 0, elems[NE], total = 0;
    void* arena = NULL;
    float* host = NULL;
    void* dev_feat[NE];
    void* dev_out[NE];
    void *dev_fresh = NULL, *dev_small = NULL;
    int e, step, fused;
    size_t i;
    FILE* fp;
    int32_t header[5];
    cudaStream_t stream;

    if (argc < 3) return 2;
    fused = argc > 3;
    memset(&cfg, 0, sizeof cfg);
    cfg.n_entries = NE;
    cfg.entries = kEntries;
    cfg.batch = B;
    cfg.max_order = M;
    cfg.dtype = SPECA_F32;
    cfg.basis = atoi(argv[2]);
    cfg.verify_entry = -1;
    cfg.device = 0;
    CK(speca_cache_arena_bytes(&cfg, &bytes) == SPECA_OK);
    CK(cudaSetDevice(0) == cudaSuccess);
    CK(cudaStreamCreate(&stream) == cudaSuccess);
    CK(cudaMalloc(&arena, bytes) == cudaSuccess);
    cfg.arena = arena;
    cfg.arena_bytes = bytes;
    CK(speca_cache_create(&cfg, &cache) == SPECA_OK);

    for (e = 0; e < NE; ++e) {
        elems[e] = (size_t)kEntries[e].tokens * (size_t)kEntries[e].dim * B;
        total += elems[e];
        CK(cudaMalloc(&dev_feat[e], elems[e] * sizeof(float)) == cudaSuccess);
        CK(cudaMalloc(&dev_out[e], elems[e] * sizeof(float)) == cudaSuccess);
    }
    host = (float*)malloc(total * sizeof(float));
    CK(host != NULL);

    /* three reference steps; features drawn entry by entry, element by element */
    g_state = 2509u;
    for (step = 0; step < 3; ++step) {
        for (e = 0; e < NE; ++e) {
            for (i = 0; i < elems[e]; ++i) host[i] = next_value();
            CK(cudaMemcpyAsync(dev_feat[e], host, elems[e] * sizeof(float), cudaMemcpyHostToDevice, stream) == cudaSuccess);
            CK(cudaStreamSynchronize(stream) == cudaSuccess); /* host[] is reused */
        }
        if (step == 2 && fused) { /* the reference step and the forecast that follows it, one pass over the tables */
            CK(speca_cache_update_forecast(cache, (const void* const*)dev_feat, kTimes[step], kMask2, kTarget, NULL,
                                           (void* const*)dev_out, NULL, NULL, stream) == SPECA_OK);
            continue;
        }
        CK(speca_cache_update(cache, (const void* const*)dev_feat, kTimes[step], step == 2 ? kMask2 : NULL, stream) == SPECA_OK);
        CK(speca_cache_commit_step(cache) == SPECA_OK);
    }

    /* speculative step: forecast everything, verify the last entry against forecast + noise */
    if (!fused) CK(speca_forecast(cache, kTarget, NULL, (void* const*)dev_out, stream) == SPECA_OK);
    {
        const size_t nv = elems[NE - 1];
        const float level[B] = {0.0f, 0.02f, 0.5f};
        float* pred = (float*)malloc(nv * sizeof(float));
        CK(pred != NULL);
        CK(cudaMemcpyAsync(pred, dev_out[NE - 1], nv * sizeof(float), cudaMemcpyDeviceToHost, stream) == cudaSuccess);
        CK(cudaStreamSynchronize(stream) == cudaSuccess);
        for (i = 0; i < nv; ++i) pred[i] += level[i / (nv / B)] * next_value();
        CK(cudaMalloc(&dev_fresh, nv * sizeof(float)) == cudaSuccess);
        CK(cudaMemcpyAsync(dev_fresh, pred, nv * sizeof(float), cudaMemcpyHostToDevice, stream) == cudaSuccess);
        CK(cudaStreamSynchronize(stream) == cudaSuccess);
        fp = fopen(argv[1], "wb");
        CK(fp != NULL);
        header[0] = B, header[1] = NE, header[2] = M, header[3] = cfg.basis, header[4] = 3;
        fwrite(header, sizeof header, 1, fp);
        for (e = 0; e < NE; ++e) {
            int32_t shape[2];
            shape[0] = (int32_t)kEntries[e].tokens, shape[1] = kEntries[e].dim;
            fwrite(shape, sizeof shape, 1, fp);
        }
        /* the verification feature, so that the harness need not redo the float addition above */
        fwrite(pred, sizeof(float), nv, fp);
        free(pred);
    }
    {
        /* small device block: err[B] f32 | spec_count[B] i32 | n_active i32 | idx[B] i32 | accept[B] | active[B] | next[B] */
        const float tau[B] = {0.05f, 0.05f, 0.05f};
        unsigned char small[4 * B + 4 * B + 4 + 4 * B + 3 * B];
        char* d;
        float* d_err;
        int32_t *d_cnt, *d_n, *d_idx;
        uint8_t *d_acc, *d_act, *d_next;
        CK(cudaMalloc(&dev_small, 256) == cudaSuccess);
        memset(small, 0, sizeof small);
        memset(small + 4 * B + 4 * B + 4 + 4 * B + B, 1, B); /* all active */
        CK(cudaMemcpyAsync(dev_small, small, sizeof small, cudaMemcpyHostToDevice, stream) == cudaSuccess);
        d = (char*)dev_small;
        d_err = (float*)d;
        d_cnt = (int32_t*)(d + 4 * B);
        d_n = (int32_t*)(d + 8 * B);
        d_idx = (int32_t*)(d + 8 * B + 4);
        d_acc = (uint8_t*)(d + 12 * B + 4);
        d_act = d_acc + B;
        d_next = d_act + B;
        CK(speca_verify_select(cache, SPECA_METRIC_L2, dev_fresh, kTarget, tau, d_act, d_next, NULL, d_err, d_acc, 4, 1,
                               d_cnt, d_idx, d_n, stream) == SPECA_OK);
        for (e = 0; e < NE; ++e) {
            CK(cudaMemcpyAsync(host, dev_out[e], elems[e] * sizeof(float), cudaMemcpyDeviceToHost, stream) == cudaSuccess);
            CK(cudaStreamSynchronize(stream) == cudaSuccess);
            fwrite(host, sizeof(float), elems[e], fp);
        }
        CK(cudaMemcpyAsync(small, dev_small, sizeof small, cudaMemcpyDeviceToHost, stream) == cudaSuccess);
        CK(cudaStreamSynchronize(stream) == cudaSuccess);
        fwrite(small, 1, 4 * B, fp);                          /* err */
        fwrite(small + 12 * B + 4, 1, B, fp);                 /* accept */
        fwrite(small + 12 * B + 4 + 2 * B, 1, B, fp);         /* next active */
        fwrite(small + 4 * B, 1, 4 * B, fp);                  /* spec_count */
        fwrite(small + 8 * B, 1, 4, fp);                      /* n_active */
        fclose(fp);
    }
    {
        speca_cache_stats_t st;
        CK(speca_cache_stats(cache, &st) == SPECA_OK);
        CK(st.verify_launches == 1 && st.select_launches == 0);
        if (fused)
            CK(st.update_launches >= 2 && st.forecast_launches == 0 && st.update_forecast_launches == 1);
        else
            CK(st.update_launches >= 3 && st.forecast_launches == 1 && st.update_forecast_launches == 0);
        CK(st.reference_steps[0] == 3 && st.reference_steps[1] == 2 && st.reference_steps[2] == 3);
    }
    CK(speca_cache_destroy(cache) == SPECA_OK);
    for (e = 0; e < NE; ++e) cudaFree(dev_feat[e]), cudaFree(dev_out[e]);
    cudaFree(dev_fresh), cudaFree(dev_small), cudaFree(arena);
    cudaStreamDestroy(stream);
    free(host);
    printf("ok\n");
    return 0;
}
