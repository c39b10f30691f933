// Evolutionary selection of low-bitwidth channel groups (Sec. 4.2, Algorithm 1): the genetic
// operators on the host (a population is a few thousand flags), the fitness of a chromosome on
// the device (the model's outputs through the mixed kernels, then the squared distance below).
#include "flexiq_internal.h"

#include <algorithm>
#include <vector>

#include "sm100_ptx.cuh"

namespace flexiq {

// ---------------------------------------------------------------------------------- device: fitness
// sum over i of (A[i] - B[i])^2 for int8 tensors, exact in int64.  (a - b)^2 = a.a - 2 a.b + b.b,
// four elements per dp4a; one 16-byte unit of each tensor per thread and step, four steps in flight.
__global__ void sq_distance_i8_kernel(const int8_t *__restrict__ A, const int8_t *__restrict__ B, long long n,
                                      unsigned long long *__restrict__ out)
{
    ptx::pdl_wait();  // A may be the previous kernel's output
    const long long units = n >> 4;
    const uint4 *a4 = reinterpret_cast<const uint4 *>(A), *b4 = reinterpret_cast<const uint4 *>(B);
    const long long step = (long long)gridDim.x * blockDim.x;
    long long acc = 0;
    for (long long base = (long long)blockIdx.x * blockDim.x + threadIdx.x; base < units; base += 4 * step) {
        uint4 va[4], vb[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const long long u = base + q * step;
            if (u < units) { va[q] = __ldg(a4 + u); vb[q] = __ldg(b4 + u); }
            else { va[q] = make_uint4(0, 0, 0, 0); vb[q] = make_uint4(0, 0, 0, 0); }
        }
        int s = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const unsigned wa[4] = {va[q].x, va[q].y, va[q].z, va[q].w}, wb[4] = {vb[q].x, vb[q].y, vb[q].z, vb[q].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int aa = __dp4a((int)wa[j], (int)wa[j], 0), bb = __dp4a((int)wb[j], (int)wb[j], 0);
                const int ab = __dp4a((int)wa[j], (int)wb[j], 0);
                s += aa + bb - 2 * ab;  // at most 4 * 255^2 per word, 16 words: far inside int32
            }
        }
        acc += s;
    }
    // the last n % 16 elements
    if (blockIdx.x == 0 && threadIdx.x < (n & 15)) {
        const int d = (int)A[(units << 4) + threadIdx.x] - (int)B[(units << 4) + threadIdx.x];
        acc += d * d;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
    __shared__ long long warp_sum[8];
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long t = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += warp_sum[w];
        if (t) atomicAdd(out, (unsigned long long)t);
    }
}

// ---------------------------------------------------------------------------------- host: operators
namespace {

constexpr uint64_t kGold = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kInitGeneration = 0xFFFFFFFFull;  // generation counter of the draws that make the seeds

inline uint64_t mix(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// 64 random bits from four counters (splitmix64 finaliser over a mix of them)
struct Draws {
    uint64_t key;
    uint64_t n = 0;
    Draws(uint64_t seed, uint64_t generation, uint64_t individual)
    {
        uint64_t z = mix(seed * kGold + kGold);
        z = mix(z ^ ((generation + 1) * 0xD1B54A32D192ED03ull));
        key = mix(z ^ ((individual + 1) * 0x8CB92BA72F3D8DD7ull));
    }
    uint64_t next() { return mix(key ^ (++n * kGold)); }
};

struct Problem {
    int n_layers;
    std::vector<int> off;  // [n_layers + 1] first flag of each layer
    const int64_t *score;
    const uint8_t *locked;  // may be NULL
    int total() const { return off.back(); }
    bool is_locked(int i) const { return locked && locked[i]; }
    uint64_t w_set(int i) const { return (1ull << 32) / (uint64_t)(1 + score[i]); }  // prefers low error scores
    uint64_t w_clear(int i) const { return (uint64_t)(1 + score[i]); }
};

// weighted choice among `cand` (index order): position of the chosen candidate in cand
template <typename W> size_t pick(const std::vector<int> &cand, W weight, Draws &d)
{
    uint64_t total = 0;
    for (int i : cand) total += weight(i);
    const uint64_t value = d.next() % total;
    uint64_t acc = 0;
    for (size_t c = 0; c < cand.size(); ++c) {
        acc += weight(cand[c]);
        if (value < acc) return c;
    }
    return cand.size() - 1;  // not reached: value < total
}

// brings the number of set flags to `target`: clears high-score flags or sets low-score ones, one at a time
void repair(uint8_t *flags, const Problem &P, long long target, Draws &d)
{
    long long total = 0;
    for (int i = 0; i < P.total(); ++i) total += flags[i];
    std::vector<int> cand;
    while (total > target) {
        cand.clear();
        for (int i = 0; i < P.total(); ++i)
            if (flags[i] && !P.is_locked(i)) cand.push_back(i);
        if (cand.empty()) break;
        flags[cand[pick(cand, [&](int i) { return P.w_clear(i); }, d)]] = 0;
        --total;
    }
    while (total < target) {
        cand.clear();
        for (int i = 0; i < P.total(); ++i)
            if (!flags[i]) cand.push_back(i);
        if (cand.empty()) break;
        flags[cand[pick(cand, [&](int i) { return P.w_set(i); }, d)]] = 1;
        ++total;
    }
}

// each set flag is cleared with probability rate_bp / 10000 and as many flags that were unset are set
// in the same layer (low scores preferred); then the total is repaired
void mutate(uint8_t *flags, const Problem &P, long long target, int rate_bp, Draws &d)
{
    std::vector<int> unset_before, cleared, cand;
    for (int l = 0; l < P.n_layers; ++l) {
        unset_before.clear();
        cleared.clear();
        for (int i = P.off[l]; i < P.off[l + 1]; ++i)
            if (!flags[i]) unset_before.push_back(i);
        for (int i = P.off[l]; i < P.off[l + 1]; ++i)
            if (flags[i] && !P.is_locked(i) && d.next() % 10000 < (uint64_t)rate_bp) cleared.push_back(i);
        for (int i : cleared) flags[i] = 0;
        cand = unset_before;
        const size_t swaps = std::min(cleared.size(), cand.size());
        for (size_t t = 0; t < swaps; ++t) {
            const size_t c = pick(cand, [&](int i) { return P.w_set(i); }, d);
            flags[cand[c]] = 1;
            cand.erase(cand.begin() + (long)c);
        }
        for (size_t t = 0; t + unset_before.size() < cleared.size(); ++t) flags[cleared[t]] = 1;  // no room: put them back
    }
    repair(flags, P, target, d);
}

int make_problem(Problem &P, int n_layers, const int32_t *groups, const int64_t *score, const uint8_t *locked)
{
    if (n_layers < 1) return set_error(FLEXIQ_ERR_INVALID_ARG, "n_layers %d must be positive", n_layers);
    if (!groups || !score) return set_error(FLEXIQ_ERR_INVALID_ARG, "groups_host or score_host is NULL");
    P.n_layers = n_layers;
    P.off.assign(1, 0);
    for (int l = 0; l < n_layers; ++l) {
        if (groups[l] < 1 || groups[l] > (1 << 20)) return set_error(FLEXIQ_ERR_INVALID_ARG, "layer %d has %d groups", l, groups[l]);
        P.off.push_back(P.off.back() + groups[l]);
    }
    for (int i = 0; i < P.total(); ++i)
        if (score[i] < 0 || score[i] >= (1ll << 31)) return set_error(FLEXIQ_ERR_INVALID_ARG, "score[%d] = %lld outside [0, 2^31)", i, (long long)score[i]);
    P.score = score;
    P.locked = locked;
    return FLEXIQ_OK;
}

}  // namespace
}  // namespace flexiq

using namespace flexiq;

extern "C" int flexiq_evo_init(int n_layers, const int32_t *groups_host, const int64_t *score_host, const uint8_t *locked_host,
                               const int32_t *per_layer_target_host, int N, uint64_t seed, uint8_t *population_host,
                               int64_t *target_out)
{
    Problem P;
    int rc = make_problem(P, n_layers, groups_host, score_host, locked_host);
    if (rc) return rc;
    if (!per_layer_target_host || !population_host) return set_error(FLEXIQ_ERR_INVALID_ARG, "per_layer_target_host or population_host is NULL");
    if (N < 1) return set_error(FLEXIQ_ERR_INVALID_ARG, "N = %d must be positive", N);
    const int total = P.total();
    // seed 0: the lowest scores of every layer (locked flags first, ties by index)
    uint8_t *greedy = population_host;
    std::fill(greedy, greedy + total, (uint8_t)0);
    std::vector<int> idx;
    for (int l = 0; l < n_layers; ++l) {
        const int g = P.off[l + 1] - P.off[l], t = per_layer_target_host[l];
        if (t < 0 || t > g) return set_error(FLEXIQ_ERR_INVALID_ARG, "layer %d: target %d outside [0, %d]", l, t, g);
        idx.resize(g);
        for (int j = 0; j < g; ++j) idx[j] = P.off[l] + j;
        std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) {
            const int la = P.is_locked(a) ? 0 : 1, lb = P.is_locked(b) ? 0 : 1;
            if (la != lb) return la < lb;
            return P.score[a] < P.score[b];
        });
        for (int j = 0; j < t; ++j) greedy[idx[j]] = 1;
        for (int j = 0; j < g; ++j)
            if (P.is_locked(idx[j])) greedy[idx[j]] = 1;
    }
    long long target = 0;
    for (int i = 0; i < total; ++i) target += greedy[i];
    // the other seeds: locked flags, then weighted draws (low scores preferred) up to the same total
    for (int c = 1; c < N; ++c) {
        uint8_t *flags = population_host + (size_t)c * total;
        for (int i = 0; i < total; ++i) flags[i] = P.is_locked(i) ? 1 : 0;
        Draws d(seed, kInitGeneration, (uint64_t)c);
        repair(flags, P, target, d);
    }
    if (target_out) *target_out = target;
    return FLEXIQ_OK;
}

extern "C" int flexiq_evo_next_generation(int n_layers, const int32_t *groups_host, const int64_t *score_host,
                                          const uint8_t *locked_host, int64_t target, int N, int k, int r, int mutation_bp,
                                          uint64_t seed, int generation, const int64_t *distance_host,
                                          const uint8_t *population_host, uint8_t *next_population_host)
{
    Problem P;
    int rc = make_problem(P, n_layers, groups_host, score_host, locked_host);
    if (rc) return rc;
    if (!distance_host || !population_host || !next_population_host)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "distance_host, population_host or next_population_host is NULL");
    if (population_host == next_population_host) return set_error(FLEXIQ_ERR_INVALID_ARG, "the next population cannot be written in place");
    if (N < 1 || k < 0 || k > N || r < 1 || r > N) return set_error(FLEXIQ_ERR_INVALID_ARG, "need 0 <= k <= N and 1 <= r <= N (N %d, k %d, r %d)", N, k, r);
    if (mutation_bp < 0 || mutation_bp > 10000) return set_error(FLEXIQ_ERR_INVALID_ARG, "mutation_bp %d outside [0, 10000]", mutation_bp);
    if (generation < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "generation %d is negative", generation);
    if (target < 0 || target > P.total()) return set_error(FLEXIQ_ERR_INVALID_ARG, "target %lld outside [0, %d]", (long long)target, P.total());
    const int total = P.total();
    // rank: ascending distance, ties by index
    std::vector<int> order(N);
    for (int i = 0; i < N; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return distance_host[a] < distance_host[b]; });
    for (int e = 0; e < k; ++e)
        std::copy(population_host + (size_t)order[e] * total, population_host + (size_t)(order[e] + 1) * total,
                  next_population_host + (size_t)e * total);
    // offspring: pairs of parents among the r fittest, one crossover point at a layer boundary
    int made = 0;
    for (int pair = 0; made < N - k; ++pair) {
        Draws d(seed, (uint64_t)generation, (uint64_t)(N + pair));
        const uint8_t *a = population_host + (size_t)order[d.next() % (uint64_t)r] * total;
        const uint8_t *b = population_host + (size_t)order[d.next() % (uint64_t)r] * total;
        const int cut = n_layers > 1 ? P.off[1 + d.next() % (uint64_t)(n_layers - 1)] : total;
        for (int child = 0; child < 2 && made < N - k; ++child, ++made) {
            uint8_t *c = next_population_host + (size_t)(k + made) * total;
            const uint8_t *left = child == 0 ? a : b, *right = child == 0 ? b : a;
            std::copy(left, left + cut, c);
            std::copy(right + cut, right + total, c + cut);
        }
    }
    for (int j = 0; j < N - k; ++j) {
        Draws d(seed, (uint64_t)generation, (uint64_t)j);
        mutate(next_population_host + (size_t)(k + j) * total, P, target, mutation_bp, d);
    }
    return FLEXIQ_OK;
}

extern "C" int flexiq_sq_distance_i8(const int8_t *A_dev, const int8_t *B_dev, int64_t n, int64_t *out_dev, void *stream)
{
    if (n < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "n = %lld is negative", (long long)n);
    if (!out_dev) return set_error(FLEXIQ_ERR_INVALID_ARG, "out_dev is NULL");
    if (n > 0 && (!A_dev || !B_dev)) return set_error(FLEXIQ_ERR_INVALID_ARG, "A_dev or B_dev is NULL");
    if ((reinterpret_cast<uintptr_t>(A_dev) | reinterpret_cast<uintptr_t>(B_dev)) & 15)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "A_dev and B_dev must be 16-byte aligned");
    int rc = check_device_sm100();
    if (rc) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    FLEXIQ_CUDA_TRY(cudaMemsetAsync(out_dev, 0, sizeof(int64_t), st));
    if (n == 0) return FLEXIQ_OK;
    int dev = 0;
    FLEXIQ_CUDA_TRY(cudaGetDevice(&dev));
    const int sms = device_sm_count(dev);
    const int threads = 256;
    long long blocks = ((n >> 4) + 4 * threads - 1) / (4 * threads);
    if (blocks < 1) blocks = 1;
    if (blocks > (long long)sms * 8) blocks = (long long)sms * 8;
    sq_distance_i8_kernel<<<(unsigned)blocks, threads, 0, st>>>(A_dev, B_dev, (long long)n, reinterpret_cast<unsigned long long *>(out_dev));
    FLEXIQ_CUDA_TRY(cudaGetLastError());
    return FLEXIQ_OK;
}
