/*
 * Driver for the sanitizer run (tests/test_sanitizers.py): compiled with -fsanitize=address,undefined
 * together with oracle/polyspec_oracle.c, it walks the oracle through ordinary and degenerate inputs
 * (empty block, -inf stretches, NaN, token out of range, the largest block), and -- when it is given the
 * path of libpolyspec.so -- calls the C ABI's host-only paths (size queries, argument checks that must
 * return before any CUDA call) with bad arguments.  Any out-of-bounds access, use of uninitialised stack,
 * signed overflow or misaligned access makes the sanitizers abort the process.
 */
#include <dlfcn.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

int pso_softmax_row(const void* row, int dtype, int64_t V, double T, double* P);
int pso_verify_level_seq(const void* p_rows, const void* q_rows, int dtype, int64_t V, int m, const int32_t* tokens,
                         const float* u_accept, float u_s, double T, int32_t* accepted_len, int32_t* next_token, double* P_at,
                         double* Q_at, double* accept_margin, double* sample_info, int32_t* used_fallback, double* scratch);
int pso_verify_chain_seq(const void* const* model_rows, const int32_t* model_nrows, int n, const int32_t* k,
                         const int32_t* draft_tokens, int bottom_len, const float* uniforms, int64_t u_level_stride, int kmax,
                         int64_t V, int dtype, double T, int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens,
                         int32_t* out_len, double* accept_margin, double* sample_info, int32_t* used_fallback, double* scratch);
int pso_argmax_row(const void* row, int dtype, int64_t V, int32_t* arg);
int pso_verify_chain_greedy_seq(const void* const* model_rows, const int32_t* model_nrows, int n, const int32_t* k,
                                const int32_t* draft_tokens, int bottom_len, int kmax, int64_t V, int dtype,
                                int32_t* accepted_len, int32_t* block_len, int32_t* out_tokens, int32_t* out_len);

static uint32_t lcg_state = 12345u;
static float rnd(void)
{
    lcg_state = lcg_state * 1664525u + 1013904223u;
    return (float)((lcg_state >> 8) + 0.5) * (1.0f / 16777216.0f);
}

static int oracle_cases(void)
{
    enum { V = 67, K = 32, N = 4 };
    int fails = 0;
    for (int round = 0; round < 40; ++round) {
        const int kk[N - 1] = {1 + round % K, 1 + (round * 7) % K, 1 + (round * 3) % K};
        int kmax = 0;
        for (int l = 0; l < N - 1; ++l) kmax = kk[l] > kmax ? kk[l] : kmax;
        int32_t nrows[N];
        float* rows[N];
        for (int i = 0; i < N; ++i) {
            nrows[i] = i < N - 1 ? kk[i] + 1 : kk[N - 2];
            rows[i] = (float*)malloc(sizeof(float) * (size_t)nrows[i] * V);
            for (int64_t e = 0; e < (int64_t)nrows[i] * V; ++e) rows[i][e] = 6.0f * rnd() - 3.0f;
        }
        if (round % 5 == 1) for (int v = 0; v < V / 2; ++v) rows[1][v] = -INFINITY;      /* a masked stretch */
        if (round % 5 == 2) rows[2][3] = NAN;
        if (round % 5 == 3) for (int v = 0; v < V; ++v) rows[0][v] = -INFINITY;          /* a row with no finite logit */
        int32_t* draft = (int32_t*)malloc(sizeof(int32_t) * (size_t)kk[N - 2]);
        for (int j = 0; j < kk[N - 2]; ++j) draft[j] = (int32_t)(rnd() * V);
        if (round % 5 == 4) draft[0] = V;                                                 /* token out of range */
        float* u = (float*)malloc(sizeof(float) * (size_t)(N - 1) * (kmax + 1));
        for (int e = 0; e < (N - 1) * (kmax + 1); ++e) u[e] = rnd();
        int32_t acc[N - 1], blk[N - 1], olen[N - 1], fb[N - 1];
        int32_t* otok = (int32_t*)malloc(sizeof(int32_t) * (size_t)(N - 1) * (kmax + 1));
        double* marg = (double*)malloc(sizeof(double) * (size_t)(N - 1) * kmax);
        double sinfo[(N - 1) * 4];
        double* scratch = (double*)malloc(sizeof(double) * 2 * V);
        const void* ptrs[N] = {rows[0], rows[1], rows[2], rows[3]};
        const int bottom = round % 3 == 0 ? kk[N - 2] / 2 : kk[N - 2];
        int st = pso_verify_chain_seq(ptrs, nrows, N, kk, draft, bottom, u, kmax + 1, kmax, V, 0, 0.9, acc, blk, otok, olen, marg,
                                      sinfo, fb, scratch);
        if (st == 0)
            for (int l = 0; l < N - 1; ++l)
                if (acc[l] < 0 || acc[l] > blk[l] || olen[l] != acc[l] + 1) ++fails;
        st = pso_verify_chain_greedy_seq(ptrs, nrows, N, kk, draft, bottom, kmax, V, 0, acc, blk, otok, olen);
        (void)st;
        /* single level with an empty block and with the whole block */
        int32_t a = 0, nx = 0, used = 0;
        double pat[K], qat[K], mg[K], si[4];
        pso_verify_level_seq(rows[2], rows[3], 0, V, 0, draft, u, u[kmax], 1.0, &a, &nx, pat, qat, mg, si, &used, scratch);
        pso_verify_level_seq(rows[2], rows[3], 0, V, kk[N - 2], draft, u, u[kmax], 1.0, &a, &nx, pat, qat, mg, si, &used, scratch);
        int32_t am = 0;
        pso_argmax_row(rows[1], 0, V, &am);
        pso_softmax_row(rows[1], 0, V, 0.5, scratch);
        for (int i = 0; i < N; ++i) free(rows[i]);
        free(draft); free(u); free(otok); free(marg); free(scratch);
    }
    /* bf16 storage: bit patterns in uint16 */
    {
        enum { V2 = 40 };
        uint16_t p[2 * V2], q[V2];
        for (int e = 0; e < 2 * V2; ++e) { float f = 4.0f * rnd() - 2.0f; uint32_t b; memcpy(&b, &f, 4); p[e] = (uint16_t)(b >> 16); }
        for (int e = 0; e < V2; ++e) { float f = 4.0f * rnd() - 2.0f; uint32_t b; memcpy(&b, &f, 4); q[e] = (uint16_t)(b >> 16); }
        int32_t tok = 7, a = 0, nx = 0, used = 0;
        float ua = 0.4f;
        double pat[1], qat[1], mg[1], si[4], scratch[2 * V2];
        if (pso_verify_level_seq(p, q, 1, V2, 1, &tok, &ua, 0.3f, 1.0, &a, &nx, pat, qat, mg, si, &used, scratch) != 0) ++fails;
        if (nx < 0 || nx >= V2) ++fails;
    }
    return fails;
}

typedef int (*ws_level_fn)(int, int, int, int, size_t*);
typedef int (*ws_chain_fn)(int, const int*, const int*, int, int, int, size_t*);
typedef int (*level_fn)(const void*, const void*, const int32_t*, const float*, const int32_t*, int, int, int, int, float, int32_t*,
                        int32_t*, float*, float*, int32_t*, void*, size_t, void*);
typedef double (*cost_fn)(int, const double*, const double*, double, double);
typedef const char* (*str_fn)(int);

static int abi_cases(const char* path)
{
    void* h = dlopen(path, RTLD_NOW);
    if (!h) { fprintf(stderr, "dlopen: %s\n", dlerror()); return 1; }
    int fails = 0;
    ws_level_fn wl = (ws_level_fn)dlsym(h, "polyspec_verify_level_workspace");
    ws_chain_fn wc = (ws_chain_fn)dlsym(h, "polyspec_verify_chain_workspace");
    level_fn lv = (level_fn)dlsym(h, "polyspec_verify_level");
    cost_fn ct = (cost_fn)dlsym(h, "polyspec_cost_total_time");
    str_fn ss = (str_fn)dlsym(h, "polyspec_status_string");
    if (!wl || !wc || !lv || !ct || !ss) return 1;
    size_t n = 0;
    const int sizes[][4] = {{1, 4, 32000, 0}, {256, 32, 152064, 1}, {0, 4, 32000, 0}, {1, 0, 8, 0}, {1, 33, 8, 0}, {1, 4, 12, 0},
                            {1, 4, 8, 9}, {1 << 30, 32, 8, 0}, {7, 3, 1 << 30, 1}};
    for (unsigned i = 0; i < sizeof sizes / sizeof sizes[0]; ++i) {
        const int st = wl(sizes[i][0], sizes[i][1], sizes[i][2], sizes[i][3], &n);
        if (i < 2 ? st != 0 : st == 0) ++fails;
    }
    if (wl(1, 4, 32000, 0, NULL) == 0) ++fails;
    const int k8[7] = {3, 3, 3, 3, 3, 3, 3}, r8[8] = {4, 4, 4, 4, 4, 4, 4, 3};
    if (wc(8, k8, r8, 5, 512, 1, &n) != 0) ++fails;
    if (wc(9, k8, r8, 5, 512, 1, &n) == 0) ++fails;         /* more models than POLYSPEC_MAX_MODELS */
    if (wc(1, k8, r8, 5, 512, 1, &n) == 0) ++fails;
    if (wc(3, NULL, r8, 5, 512, 1, &n) == 0) ++fails;
    /* argument checks of a verify call: every one must return before CUDA is touched */
    static float fake[64];
    int32_t tok[4] = {0, 1, 2, 3}, out[2];
    if (lv(NULL, fake, tok, fake, NULL, 1, 4, 8, 0, 1.0f, out, out + 1, NULL, NULL, NULL, fake, 1 << 20, NULL) == 0) ++fails;
    if (lv(fake, fake, tok, fake, NULL, 1, 4, 8, 0, 0.0f, out, out + 1, NULL, NULL, NULL, fake, 1 << 20, NULL) == 0) ++fails;
    if (lv(fake, fake, tok, fake, NULL, 1, 4, 8, 0, NAN, out, out + 1, NULL, NULL, NULL, fake, 1 << 20, NULL) == 0) ++fails;
    if (lv(fake, fake, tok, fake, NULL, 1, 4, 8, 0, 1.0f, out, NULL, NULL, NULL, NULL, fake, 1 << 20, NULL) == 0) ++fails;
    if (lv(fake, fake, tok, fake, NULL, 1, 4, 8, 0, 1.0f, out, out + 1, NULL, NULL, NULL, NULL, 0, NULL) == 0) ++fails;
    if (lv((char*)fake + 4, fake, tok, fake, NULL, 1, 4, 8, 0, 1.0f, out, out + 1, NULL, NULL, NULL, fake, 1 << 20, NULL) == 0) ++fails;
    const double T[3] = {10.0, 3.0, 1.0}, Ls[2] = {4.0, 2.0};
    if (!(ct(3, T, Ls, 1.0, 100.0) > 0.0)) ++fails;
    if (!isnan(ct(1, T, Ls, 1.0, 100.0))) ++fails;
    for (int s = -2; s < 12; ++s) if (!ss(s)) ++fails;
    dlclose(h);
    return fails;
}

int main(int argc, char** argv)
{
    int fails = oracle_cases();
    if (argc > 1) fails += abi_cases(argv[1]);
    printf("sanitize_driver: %d failed checks\n", fails);
    return fails ? 1 : 0;
}
