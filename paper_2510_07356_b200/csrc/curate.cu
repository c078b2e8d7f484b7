// Curation arithmetic of the ConCuR pipeline over a table of generation records: Eq. (1)-(3),
// the selection rules (a) and (b), the four ablation selections, the length / speedup
// correlation and the difficulty bins.  Three small stream-ordered kernels: one thread per task
// for everything that is local to a task (with block-reduced counts and sums), one thread per
// task and selection for the rank among all tasks (a counting rank: exact, deterministic, tie
// order by task index, no scratch memory), one thread for the derived statistics.
#include "../../include/concur_attn.h"
#include "../../include/concur_curate.h"

#include <cuda_runtime.h>
#include <math.h>

namespace {

constexpr int kThreads = 256;
constexpr int kSums = 15;          // stats 0 .. 14 are sums

// Sums of one block into the global statistics (float64 atomics: every term is an integer or a
// float32 value, so only the order of the last few additions can differ between runs).
__device__ void block_add(double (&v)[kSums], double* stats) {
    __shared__ double sm[kThreads / 32][kSums];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    #pragma unroll
    for (int k = 0; k < kSums; ++k) {
        double x = v[k];
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        if (lane == 0) sm[warp][k] = x;
    }
    __syncthreads();
    if (threadIdx.x < kSums) {
        double x = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) x += sm[w][threadIdx.x];
        if (x != 0.0) atomicAdd(stats + threadIdx.x, x);
    }
}

__global__ void __launch_bounds__(kThreads)
curate_tasks_kernel(concur_curate_params_t prm, const uint8_t* __restrict__ correct, const float* __restrict__ t_torch,
                    const float* __restrict__ t_kernel, const int32_t* __restrict__ length,
                    const float* __restrict__ sample_key, float* __restrict__ speedup, int32_t* __restrict__ rule_a,
                    uint8_t* __restrict__ rule_b, int32_t* __restrict__ pick, uint8_t* __restrict__ difficulty,
                    double* stats) {
    const int i = blockIdx.x * kThreads + threadIdx.x;
    const int N = prm.num_tasks, M = prm.gens;
    double v[kSums];
    #pragma unroll
    for (int k = 0; k < kSums; ++k) v[k] = 0.0;
    if (i < N) {
        const int64_t base = (int64_t)i * M;
        int shortest = 0, p_rand = -1, p_long = -1, p_short = -1, p_fast = -1;
        float best = 0.f, sp_shortest = 0.f, sp_fast = 0.f, key_rand = 0.f;
        int32_t len_shortest = 0, len_long = 0, len_short = 0;
        bool shortest_correct = false;
        int64_t len_sum = 0;
        for (int j = 0; j < M; ++j) {
            const bool ok = correct[base + j] != 0;
            const int32_t L = length[base + j];
            // Eq. (1): an IEEE float32 quotient, so that every comparison below is decided on the
            // same value as in a float32 reference
            const float sp = ok ? __fdiv_rn(t_torch[base + j], t_kernel[base + j]) : 0.f;
            speedup[base + j] = sp;
            const bool b = sp > prm.rule_b_speedup;
            rule_b[base + j] = b ? 1 : 0;
            len_sum += L;
            best = fmaxf(best, sp);
            if (j == 0 || L < len_shortest) { shortest = j; len_shortest = L; sp_shortest = sp; shortest_correct = ok; }
            if (ok) {
                const float key = sample_key[base + j];
                if (p_rand < 0 || key > key_rand) { p_rand = j; key_rand = key; }
                if (p_long < 0 || L > len_long) { p_long = j; len_long = L; }
                if (p_short < 0 || L < len_short) { p_short = j; len_short = L; }
                if (p_fast < 0 || sp > sp_fast) { p_fast = j; sp_fast = sp; }
                const double x = (double)L, y = (double)sp;
                v[CONCUR_STAT_CORRECT] += 1.0; v[CONCUR_STAT_N] += 1.0;
                v[CONCUR_STAT_SX] += x; v[CONCUR_STAT_SY] += y;
                v[CONCUR_STAT_SXX] += x * x; v[CONCUR_STAT_SYY] += y * y; v[CONCUR_STAT_SXY] += x * y;
            }
            if (b) v[CONCUR_STAT_RULE_B] += 1.0;
            if (j == 0) {
                if (sp > prm.fast_p) v[CONCUR_STAT_FAST_FIRST_COUNT] += 1.0;
                if (ok) v[CONCUR_STAT_EXEC_FIRST_COUNT] += 1.0;
            }
        }
        // rule (a): the shortest generation, if it is correct and nothing is faster
        const bool a = shortest_correct && sp_shortest >= best;
        rule_a[i] = a ? shortest : -1;
        pick[0 * (int64_t)N + i] = p_rand;
        pick[1 * (int64_t)N + i] = p_long;
        pick[2 * (int64_t)N + i] = p_short;
        pick[3 * (int64_t)N + i] = p_fast;
        difficulty[i] = len_sum < (int64_t)M * prm.easy_below ? 0 : (len_sum > (int64_t)M * prm.hard_above ? 2 : 1);
        if (a) v[CONCUR_STAT_RULE_A] += 1.0;
        if (p_fast >= 0) v[CONCUR_STAT_TASKS_CORRECT] += 1.0;
        if (best > prm.fast_p) v[CONCUR_STAT_FAST_BEST_COUNT] += 1.0;
        v[CONCUR_STAT_LENGTH_SUM] += (double)len_sum;
    }
    block_add(v, stats);
}

// The key by which selection s ranks task j, as a double in "larger ranks first" form (exact for
// int32 lengths and float32 keys); `valid` is false for a task without a correct generation.
__device__ __forceinline__ double selection_key(int s, int j, int N, int M, const int32_t* pick, const int32_t* length,
                                                const float* speedup, const float* task_key, bool* valid) {
    const int32_t pj = pick[(int64_t)s * N + j];
    *valid = pj >= 0;
    if (pj < 0) return 0.0;
    switch (s) {
        case CONCUR_SEL_RANDOM: return (double)task_key[j];
        case CONCUR_SEL_MAX_LENGTH: return (double)length[(int64_t)j * M + pj];
        case CONCUR_SEL_MIN_LENGTH: return -(double)length[(int64_t)j * M + pj];
        default: return (double)speedup[(int64_t)j * M + pj];
    }
}

__global__ void __launch_bounds__(kThreads)
curate_rank_kernel(concur_curate_params_t prm, const int32_t* __restrict__ pick, const int32_t* __restrict__ length,
                   const float* __restrict__ speedup, const float* __restrict__ task_key, uint8_t* __restrict__ keep) {
    __shared__ double keys[kThreads];
    __shared__ uint8_t valids[kThreads];
    const int s = blockIdx.y;
    const int N = prm.num_tasks, M = prm.gens;
    const int i = blockIdx.x * kThreads + threadIdx.x;
    bool valid_i = false;
    const double key_i = i < N ? selection_key(s, i, N, M, pick, length, speedup, task_key, &valid_i) : 0.0;
    int32_t rank = 0;
    for (int base = 0; base < N; base += kThreads) {
        const int j = base + threadIdx.x;
        bool vj = false;
        keys[threadIdx.x] = j < N ? selection_key(s, j, N, M, pick, length, speedup, task_key, &vj) : 0.0;
        valids[threadIdx.x] = vj ? 1 : 0;
        __syncthreads();
        const int lim = min(kThreads, N - base);
        for (int t = 0; t < lim; ++t) {
            const double kj = keys[t];
            // tasks that come before task i: a larger key, or the same key and a lower index
            if (valids[t] && (kj > key_i || (kj == key_i && base + t < i))) ++rank;
        }
        __syncthreads();
    }
    if (i < N) keep[(int64_t)s * N + i] = (valid_i && rank < prm.top_k) ? 1 : 0;
}

__global__ void curate_finish_kernel(concur_curate_params_t prm, double* stats) {
    const double NM = (double)prm.num_tasks * prm.gens;
    stats[CONCUR_STAT_ARL] = stats[CONCUR_STAT_LENGTH_SUM] / NM;
    stats[CONCUR_STAT_FAST_FIRST] = stats[CONCUR_STAT_FAST_FIRST_COUNT] / prm.num_tasks;
    stats[CONCUR_STAT_FAST_BEST] = stats[CONCUR_STAT_FAST_BEST_COUNT] / prm.num_tasks;
    const double n = stats[CONCUR_STAT_N];
    double r = nan("");
    if (n >= 2.0) {
        const double sx = stats[CONCUR_STAT_SX], sy = stats[CONCUR_STAT_SY];
        const double cov = stats[CONCUR_STAT_SXY] - sx * sy / n;
        const double vx = stats[CONCUR_STAT_SXX] - sx * sx / n;
        const double vy = stats[CONCUR_STAT_SYY] - sy * sy / n;
        if (vx * vy > 0.0) r = cov / sqrt(vx * vy);      // a constant column: undefined, NaN
    }
    stats[CONCUR_STAT_PEARSON_R] = r;
}

}  // namespace

extern "C" int concur_curate(const concur_curate_params_t* prm, const uint8_t* correct, const float* t_torch,
                             const float* t_kernel, const int32_t* length, const float* sample_key,
                             const float* task_key, float* speedup, int32_t* rule_a, uint8_t* rule_b, int32_t* pick,
                             uint8_t* keep, uint8_t* difficulty, double* stats, void* cuda_stream) {
    if (!prm || prm->reserved != 0) return CONCUR_ERR_INVALID_ARG;
    if (prm->num_tasks < 1 || prm->gens < 1 || prm->gens > 32 || prm->top_k < 0) return CONCUR_ERR_INVALID_ARG;
    if ((int64_t)prm->num_tasks * prm->gens >= (int64_t)1 << 31) return CONCUR_ERR_INVALID_ARG;
    if (!correct || !t_torch || !t_kernel || !length || !sample_key || !task_key || !speedup || !rule_a || !rule_b ||
        !pick || !keep || !difficulty || !stats)
        return CONCUR_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(stats, 0, sizeof(double) * CONCUR_CURATE_NUM_STATS, stream) != cudaSuccess) {
        cudaGetLastError();
        return CONCUR_ERR_CUDA;
    }
    const int blocks = (prm->num_tasks + kThreads - 1) / kThreads;
    curate_tasks_kernel<<<blocks, kThreads, 0, stream>>>(*prm, correct, t_torch, t_kernel, length, sample_key, speedup,
                                                         rule_a, rule_b, pick, difficulty, stats);
    curate_rank_kernel<<<dim3(blocks, CONCUR_NUM_SELECTIONS), kThreads, 0, stream>>>(*prm, pick, length, speedup,
                                                                                    task_key, keep);
    curate_finish_kernel<<<1, 1, 0, stream>>>(*prm, stats);
    if (cudaGetLastError() != cudaSuccess) return CONCUR_ERR_CUDA;
    return CONCUR_OK;
}
