// CUDA twin of logits.py: writes the same bits.  Input generation only -- no part of the decoding method.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__host__ __device__ inline uint64_t mix(uint64_t x) {   // splitmix64 output function
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

constexpr uint64_t kBoostSalt = 0xB0057B0057B0057Bull;
constexpr int kBoostP16 = 19661;
constexpr int kEos = 2;

__device__ inline uint16_t bf16_rne(float x) {
    uint32_t b = __float_as_uint(x);
    return (uint16_t)((b + 0x7FFFu + ((b >> 16) & 1u)) >> 16);
}

__global__ void gen_kernel(void* __restrict__ out, int bf16, int R, int V, int k, int64_t stride, uint64_t base_key,
                           int step, const int64_t* __restrict__ sent_ids, const int32_t* __restrict__ last_token,
                           const uint64_t* __restrict__ met_mask, const int32_t* __restrict__ ctok,
                           const int32_t* __restrict__ ncon, const float* __restrict__ table,
                           const float* __restrict__ mu, float sigma, int zipf, int boost,
                           const int32_t* __restrict__ end_step, float eos_late) {
    const int r = blockIdx.y;
    const int quad = blockIdx.x * blockDim.x + threadIdx.x;
    if (quad * 4 >= V) return;
    const int b = r / k;
    const uint64_t key = mix(mix(mix(base_key + (uint64_t)step) + (uint64_t)sent_ids[b]) + (uint64_t)(int64_t)last_token[r]);
    int boost_tok = -1;
    if (boost && (int)(mix(key ^ kBoostSalt) & 0xFFFFull) < kBoostP16) {
        const uint64_t inv = ~met_mask[r];
        const int j = inv ? __ffsll((long long)inv) - 1 : 64;
        if (j < ncon[b]) boost_tok = ctok[b * 64 + j];
    }
    const bool late = zipf && step >= end_step[b];
    const uint64_t hq = mix(key + (uint64_t)quad);
#pragma unroll
    for (int l = 0; l < 4; ++l) {
        const int w = quad * 4 + l;
        if (w >= V) break;
        const float z = table[(hq >> (16 * l)) & 0xFFFFull];
        float x = __fadd_rn(__fmul_rn(sigma, z), (late && w == kEos) ? eos_late : mu[w]);
        if (w == boost_tok) x = __fadd_rn(x, 4.0f);
        if (bf16) ((uint16_t*)out)[(int64_t)r * stride + w] = bf16_rne(x);
        else ((float*)out)[(int64_t)r * stride + w] = x;
    }
}

}  // namespace

extern "C" int synth_gen_logits(void* out, int bf16, int R, int V, int k, int64_t stride, uint64_t base_key, int step,
                                const int64_t* sent_ids, const int32_t* last_token, const uint64_t* met_mask,
                                const int32_t* ctok, const int32_t* ncon, const float* table, const float* mu,
                                float sigma, int zipf, int boost, const int32_t* end_step, float eos_late,
                                void* stream) {
    const int threads = 256;
    dim3 grid(((V + 3) / 4 + threads - 1) / threads, R);
    gen_kernel<<<grid, threads, 0, (cudaStream_t)stream>>>(out, bf16, R, V, k, stride, base_key, step, sent_ids,
                                                          last_token, met_mask, ctok, ncon, table, mu, sigma, zipf,
                                                          boost, end_step, eos_late);
    return (int)cudaGetLastError();
}
