// Seeded synthetic-input generator: weights, per-sublayer scales and prompts.
//
// This module produces DATA only. It holds none of the decoder's, the cosine
// rule's or ADMG's arithmetic; both the CPU oracle and the CUDA library receive
// its output as plain buffers.
//
// Every value is a pure function of (seed, tensor_id, element index), so
// generation is order independent and can run on any number of threads:
//   key   = mix64(seed * GOLDEN + tensor_id)
//   r     = mix64(key + pair_index * GOLDEN)           (one draw per PAIR of elements)
//   u1,u2 = the high / low 32 bits of r mapped to (0,1)
//   z0,z1 = Box-Muller(u1,u2)                           (element 2j gets z0, 2j+1 gets z1)
// mix64 is the SplitMix64 output function (Steele, Lea, Flood 2014).
#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>

namespace {

constexpr uint64_t GOLDEN = 0x9E3779B97F4A7C15ull;

inline uint64_t mix64(uint64_t z) {
    z += GOLDEN;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

inline uint64_t stream_key(uint64_t seed, uint64_t tensor_id) { return mix64(seed * GOLDEN + tensor_id); }

inline double unit_open(uint32_t bits) { return ((double)bits + 0.5) * (1.0 / 4294967296.0); }

inline void normal_pair(uint64_t key, uint64_t pair, double& z0, double& z1) {
    uint64_t r = mix64(key + pair * GOLDEN);
    double u1 = unit_open((uint32_t)(r >> 32));
    double u2 = unit_open((uint32_t)r);
    double rad = std::sqrt(-2.0 * std::log(u1));
    double ang = 6.283185307179586476925286766559 * u2;
    z0 = rad * std::cos(ang);
    z1 = rad * std::sin(ang);
}

// float -> bfloat16 bits, round to nearest even (inputs are finite).
inline uint16_t to_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

}  // namespace

extern "C" {

// out[i] = bf16( (mean + std * z_i) * scale ),  i in [0, n)
void synth_normal_bf16(uint16_t* out, size_t n, uint64_t seed, uint64_t tensor_id, double mean, double std,
                       double scale) {
    const uint64_t key = stream_key(seed, tensor_id);
    const size_t pairs = (n + 1) / 2;
#pragma omp parallel for schedule(static)
    for (size_t j = 0; j < pairs; ++j) {
        double z0, z1;
        normal_pair(key, j, z0, z1);
        out[2 * j] = to_bf16((float)((mean + std * z0) * scale));
        if (2 * j + 1 < n) out[2 * j + 1] = to_bf16((float)((mean + std * z1) * scale));
    }
}

// out[i] = lo + (hi - lo) * u_i, u_i uniform in (0,1)
void synth_uniform_f64(double* out, size_t n, uint64_t seed, uint64_t tensor_id, double lo, double hi) {
    const uint64_t key = stream_key(seed, tensor_id);
    for (size_t i = 0; i < n; ++i) {
        uint64_t r = mix64(key + i * GOLDEN);
        double u = ((double)(r >> 11) + 0.5) * (1.0 / 9007199254740992.0);
        out[i] = lo + (hi - lo) * u;
    }
}

// out[i] uniform integer in [0, bound)
void synth_uniform_i32(int32_t* out, size_t n, uint64_t seed, uint64_t tensor_id, int32_t bound) {
    const uint64_t key = stream_key(seed, tensor_id);
    for (size_t i = 0; i < n; ++i) {
        uint64_t r = mix64(key + i * GOLDEN);
        out[i] = (int32_t)(((r >> 32) * (uint64_t)bound) >> 32);
    }
}

}  // extern "C"
