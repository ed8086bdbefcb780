/*
 * A second CPU baseline: the same scatter-sum as dst_oracle.c, in fp32 and on
 * every host core.  TEST INFRASTRUCTURE ONLY, like the oracle beside it: the
 * benchmark times it as "what a plain multi-core CPU loop does", a test pins
 * it against the fp64 oracle, and nothing on the product path may call it.
 *
 * The operation is the one of the paper's Section 4 (Listing 1) followed by
 * the reduction of Algorithm 1:
 *
 *   out[v, c] = dense_in[v, c] (or 0) + sum over slices r, rows i with
 *                                        indices_r[i] == v of values_r[i, c]
 *
 * Parallel over disjoint column blocks: thread t owns columns [c0_t, c1_t) of
 * every output row, walks all input rows in the order given and adds its part
 * of each.  No two threads touch the same output element, so there are no
 * atomics, no sorting and no locks; every output element is summed in input
 * order in fp32 (bf16 values are widened exactly; a bf16 output is rounded
 * once at the end from the fp32 sum).
 *
 * Pin: tests/test_cpu_threads.py compares it with the fp64 oracle (fp32
 * tolerance, bit-exact on small-integer data and for the row counters).
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    const void* indices; /* int32 or int64, n_rows entries */
    const void* values;  /* float or bf16 bits (uint16), n_rows * d entries, row-major */
    int64_t n_rows;
} cpu_slice_t;

typedef struct {
    const cpu_slice_t* slices;
    int32_t R;
    int index_is_i64, value_is_bf16, out_is_bf16;
    int64_t d, vocab, c0, c1;
    const void* dense_in;
    void* out;      /* [vocab*d] float or bf16 bits */
    float* scratch; /* [vocab*d] fp32 sums when the output is bf16, else NULL (out is used) */
    int64_t n_bad;  /* counted by the thread that owns column 0 */
} job_t;

static float bf16_to_float(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* fp32 -> bf16, nearest, ties to even */
static uint16_t float_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0u; /* NaN */
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static void* run_block(void* arg) {
    job_t* j = (job_t*)arg;
    const int64_t d = j->d, w = j->c1 - j->c0;
    float* sum = j->out_is_bf16 ? j->scratch : (float*)j->out;
    for (int64_t v = 0; v < j->vocab; ++v) {
        float* o = sum + v * d + j->c0;
        if (!j->dense_in) {
            for (int64_t c = 0; c < w; ++c) o[c] = 0.0f;
        } else if (j->out_is_bf16) {
            const uint16_t* s = (const uint16_t*)j->dense_in + v * d + j->c0;
            for (int64_t c = 0; c < w; ++c) o[c] = bf16_to_float(s[c]);
        } else {
            const float* s = (const float*)j->dense_in + v * d + j->c0;
            for (int64_t c = 0; c < w; ++c) o[c] = s[c];
        }
    }
    int64_t bad = 0;
    for (int32_t r = 0; r < j->R; ++r) {
        const cpu_slice_t* s = &j->slices[r];
        for (int64_t i = 0; i < s->n_rows; ++i) {
            const int64_t v = j->index_is_i64 ? ((const int64_t*)s->indices)[i]
                                              : (int64_t)((const int32_t*)s->indices)[i];
            if (v < 0 || v >= j->vocab) { ++bad; continue; }
            float* o = sum + v * d + j->c0;
            if (j->value_is_bf16) {
                const uint16_t* row = (const uint16_t*)s->values + i * d + j->c0;
                for (int64_t c = 0; c < w; ++c) o[c] += bf16_to_float(row[c]);
            } else {
                const float* row = (const float*)s->values + i * d + j->c0;
                for (int64_t c = 0; c < w; ++c) o[c] += row[c];
            }
        }
    }
    if (j->out_is_bf16) {
        for (int64_t v = 0; v < j->vocab; ++v) {
            const float* a = sum + v * d + j->c0;
            uint16_t* o = (uint16_t*)j->out + v * d + j->c0;
            for (int64_t c = 0; c < w; ++c) o[c] = float_to_bf16(a[c]);
        }
    }
    j->n_bad = bad;
    return NULL;
}

/*
 * n_threads: column blocks / threads to use (clamped to [1, d]).
 * scratch  : [vocab*d] floats, needed only when out_is_bf16.
 * returns the number of threads used, or -1 on a bad argument.
 */
int dst_cpu_threads_densify(const cpu_slice_t* slices, int32_t R, int index_is_i64, int value_is_bf16,
                            int out_is_bf16, int64_t d, int64_t vocab, const void* dense_in, void* out,
                            float* scratch, int n_threads, int64_t* n_bad) {
    if (R < 0 || d < 0 || vocab < 0 || (R > 0 && !slices) || (vocab * d > 0 && !out)) return -1;
    if (out_is_bf16 && vocab * d > 0 && !scratch) return -1;
    for (int32_t r = 0; r < R; ++r) if (slices[r].n_rows < 0) return -1;
    if (n_bad) *n_bad = 0;
    if (d == 0) return 0;
    if (n_threads < 1) n_threads = 1;
    if ((int64_t)n_threads > d) n_threads = (int)d;
    job_t* jobs = (job_t*)calloc((size_t)n_threads, sizeof(job_t));
    pthread_t* th = (pthread_t*)calloc((size_t)n_threads, sizeof(pthread_t));
    if (!jobs || !th) { free(jobs); free(th); return -1; }
    for (int t = 0; t < n_threads; ++t) {
        job_t* j = &jobs[t];
        j->slices = slices; j->R = R;
        j->index_is_i64 = index_is_i64; j->value_is_bf16 = value_is_bf16; j->out_is_bf16 = out_is_bf16;
        j->d = d; j->vocab = vocab;
        j->c0 = d * t / n_threads; j->c1 = d * (t + 1) / n_threads;
        j->dense_in = dense_in; j->out = out; j->scratch = scratch;
    }
    int started = 0;
    for (int t = 1; t < n_threads; ++t) {
        if (pthread_create(&th[t], NULL, run_block, &jobs[t]) != 0) break;
        started = t;
    }
    run_block(&jobs[0]);
    for (int t = started + 1; t < n_threads; ++t) run_block(&jobs[t]); /* threads that could not be created */
    for (int t = 1; t <= started; ++t) pthread_join(th[t], NULL);
    if (n_bad) *n_bad = jobs[0].n_bad;
    free(jobs); free(th);
    return n_threads;
}
