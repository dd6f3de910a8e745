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

}  // namespace maaso
