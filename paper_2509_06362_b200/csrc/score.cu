// Composite serving score of Sec. IV-D from the integer result records, in IEEE double with
// explicitly rounded operations (no fused multiply-add), so that it reproduces a plain
// sequential evaluation bit for bit.
#include "common.cuh"

namespace maaso {

__global__ void score_kernel(const maaso_result* res, uint64_t n, maaso_score_params p, double* out) {
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint4 a = reinterpret_cast<const uint4*>(res + i)[0];  // status, counted, served, hit
    const uint4 d = reinterpret_cast<const uint4*>(res + i)[3];  // .., .., sum_ttft
    const uint4 m = reinterpret_cast<const uint4*>(res + i)[5];  // max_e2e, makespan
    const uint4 t = reinterpret_cast<const uint4*>(res + i)[6];  // tokens, checksum
    if (a.x != 0) { out[i] = -1.0; return; }
    const uint32_t n_counted = a.y, n_served = a.z, n_hit = a.w;
    const int64_t sum_ttft = (int64_t)(((uint64_t)d.w << 32) | d.z);
    const int64_t makespan = (int64_t)(((uint64_t)m.w << 32) | m.z);
    const uint64_t tokens = ((uint64_t)t.y << 32) | t.x;
    double phis = 0.0, phit = 0.0, phil = 0.0;
    if (n_counted > 0) phis = __ddiv_rn((double)n_hit, (double)n_counted);           // Phi_S^n: SLO satisfaction ratio
    if (n_served > 0 && makespan > 0) {
        const double thr = __ddiv_rn((double)tokens, __dmul_rn((double)makespan, 1e-6));  // tokens per second
        phit = __ddiv_rn(thr < p.gamma_t ? thr : p.gamma_t, p.gamma_t);                   // Phi_T^n
    }
    if (n_served > 0) {
        const double lat = __dmul_rn(__ddiv_rn((double)sum_ttft, (double)n_served), 1e-6);  // mean time to first token, s
        double room = __dadd_rn(p.gamma_l, -lat);
        if (room < 0.0) room = 0.0;
        phil = __ddiv_rn(room, p.gamma_l);                                                // Phi_L^n
    }
    const double x = __dmul_rn(p.alpha, phis);
    const double y = __dmul_rn(p.beta, phit);
    const double z = __dmul_rn(__dadd_rn(1.0, -p.beta), phil);
    out[i] = __dadd_rn(__dadd_rn(x, y), z);
}

cudaError_t launch_score(const maaso_result* res, uint64_t n, const maaso_score_params& p, double* out,
                         cudaStream_t stream) {
    if (n) score_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(res, n, p, out);
    return cudaGetLastError();
}

// Upper edge (microseconds) of a histogram bin of ttft_bin; the last bin is open.
__device__ __forceinline__ int64_t ttft_bin_upper(uint32_t b) {
    if (b == 0) return 1023;
    if (b >= (uint32_t)(MAASO_TTFT_BINS - 1)) return INT64_MAX;
    const uint32_t e = 10u + (b - 1u) / 2u, h = (b - 1u) & 1u;
    return ((int64_t)1 << e) + (int64_t)(h + 1u) * ((int64_t)1 << (e - 1)) - 1;
}

struct PermilleList {
    uint32_t v[16];
};

// One thread per candidate: cumulative counts over the 64 bins, one pass per requested rank.
__global__ void ttft_percentile_kernel(const uint32_t* hist, uint64_t n, PermilleList pm, uint32_t n_p, int64_t* out) {
    const uint64_t c = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n) return;
    const uint32_t* h = hist + c * MAASO_TTFT_BINS;
    uint64_t total = 0;
    for (int b = 0; b < MAASO_TTFT_BINS; b++) total += h[b];
    for (uint32_t j = 0; j < n_p; j++) {
        int64_t r = -1;
        if (total > 0) {
            uint64_t target = ((uint64_t)pm.v[j] * total + 999u) / 1000u;
            if (target < 1) target = 1;
            uint64_t cum = 0;
            for (int b = 0; b < MAASO_TTFT_BINS; b++) {
                cum += h[b];
                if (cum >= target) { r = ttft_bin_upper((uint32_t)b); break; }
            }
        }
        out[c * n_p + j] = r;
    }
}

cudaError_t launch_ttft_percentiles(const uint32_t* hist, uint64_t n, const uint32_t* permille, uint32_t n_p,
                                    int64_t* out, cudaStream_t stream) {
    PermilleList pm;
    for (uint32_t j = 0; j < 16; j++) pm.v[j] = j < n_p ? permille[j] : 0;
    if (n) ttft_percentile_kernel<<<(unsigned)((n + 127) / 128), 128, 0, stream>>>(hist, n, pm, n_p, out);
    return cudaGetLastError();
}

}  // namespace maaso
