// Optional rotary position embedding (the paper omits positional terms "for clarity"; Eq. 2 as
// printed has none and the library's default is none).  LLaMA convention, "rotate half": inside a
// head, components i and i + dh/2 are rotated by pos * theta^(-2i/dh); pos = position - 1.  The query
// of position p uses p - 1, the key made from the state at position j uses j - 1 (true or draft /
// predicted state alike), so scores depend on p - j only.  Values are not rotated.
//
// The projections write Q and K unrotated; these kernels rotate them in place afterwards, from a
// table of (cos, sin) per (position, i) that is built once in double precision, so large angles
// keep full accuracy.  The backward applies the opposite rotation to dQ and dK.
#include "kernels.h"

namespace beagle {

namespace {

__global__ void __launch_bounds__(256) rope_table_kernel(double log2_theta, int dh, int npos, float2* __restrict__ table) {
    const int half = dh >> 1;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)npos * half) return;
    const int pos = (int)(idx / half), i = (int)(idx % half);
    const double freq = exp2(-2.0 * (double)i / (double)dh * log2_theta);
    double s, c;
    sincos((double)pos * freq, &s, &c);
    table[idx] = make_float2((float)c, (float)s);
}

// One head's vector at `v` (dh elements), rotated in place by the table row `t`; sgn = +1 forward, -1 inverse.
template <typename T>
__device__ __forceinline__ void rotate_head(T* v, const float2* __restrict__ t, int half, float sgn, int lane, int nlanes) {
    for (int i = lane; i < half; i += nlanes) {
        const float2 cs = t[i];
        const float a = to_float<T>(v[i]), b = to_float<T>(v[i + half]);
        const float sn = sgn * cs.y;
        v[i] = from_float<T>(a * cs.x - b * sn);
        v[i + half] = from_float<T>(b * cs.x + a * sn);
    }
}

// Rows of a dense [rows, H*dh] matrix; row r sits at position pos_base + r % S.  One warp per (row, head).
template <typename T>
__global__ void __launch_bounds__(256) rope_rows_kernel(T* __restrict__ x, long long pairs, int H, int dh, int S, int pos_base, float sgn,
                                                       const float2* __restrict__ table) {
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (w >= pairs) return;
    const long long row = w / H;
    const int pos = pos_base + (int)(row % S);
    rotate_head<T>(x + w * dh, table + (size_t)pos * (dh >> 1), dh >> 1, sgn, threadIdx.x & 31, 32);
}

// Serve-time step: blockIdx.y < Hq rotates head y of query row b (position qpos[b]); the other
// blockIdx.y rotate K/V head y - Hq of the key row just appended for row b at cache row app[b]
// (position kpos[b]; app[b] < 0: nothing was appended).  One warp per CTA.
template <typename T>
__global__ void __launch_bounds__(32) rope_serve_kernel(T* __restrict__ q, int nq, int Hq, T* __restrict__ kcache, int nk, int Hkv, int dh, int cap,
                                                       const RowMap slot, const RowMap app, const RowMap qpos, const RowMap kpos,
                                                       const float2* __restrict__ table) {
    pdl_wait();
    pdl_launch_dependents();
    const int b = blockIdx.x, y = blockIdx.y, half = dh >> 1;
    if (y < Hq) {
        if (b < nq) rotate_head<T>(q + ((size_t)b * Hq + y) * dh, table + (size_t)qpos.idx[b] * half, half, 1.f, threadIdx.x, 32);
    } else if (b < nk && app.idx[b] >= 0 && BEAGLE_IN_BOUNDS(app.idx[b] < cap && BEAGLE_SLOT_OK(slot.idx[b]))) {
        T* row = kcache + (((size_t)slot.idx[b] * Hkv + (y - Hq)) * cap + app.idx[b]) * dh;
        rotate_head<T>(row, table + (size_t)kpos.idx[b] * half, half, 1.f, threadIdx.x, 32);
    }
}

__device__ __forceinline__ int seq_of(const SeqRows& rows, int r) {
    int b = 0;
    while (b + 1 < rows.n && r >= rows.row_start[b + 1]) ++b;
    return b;
}

// Key rows appended by a prefill: packed row r of sequence s went to cache row pos_start[s] + (r - row_start[s]),
// which is also its position.  One warp per (row, K/V head).
template <typename T>
__global__ void __launch_bounds__(256) rope_cache_rows_kernel(T* __restrict__ kcache, long long pairs, int Hkv, int dh, int cap, const SeqRows rows,
                                                             const float2* __restrict__ table) {
    const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (w >= pairs) return;
    const int r = (int)(w / Hkv), h = (int)(w % Hkv);
    const int s = seq_of(rows, r);
    const int pos = rows.pos_start[s] + (r - rows.row_start[s]);
    if (!BEAGLE_IN_BOUNDS(pos >= 0 && pos < cap && BEAGLE_SLOT_OK(rows.slot[s]))) return;
    rotate_head<T>(kcache + (((size_t)rows.slot[s] * Hkv + h) * cap + pos) * dh, table + (size_t)pos * (dh >> 1), dh >> 1, 1.f,
                   threadIdx.x & 31, 32);
}

}  // namespace

int launch_rope_table(float theta, int dh, int npos, float* table, cudaStream_t stream) {
    if (npos <= 0) return 0;
    const long long n = (long long)npos * (dh / 2);
    rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(log2((double)theta), dh, npos, reinterpret_cast<float2*>(table));
    return 1;
}

int launch_rope_rows(int dtype, void* x, long long rows, int H, int dh, int S, int pos_base, int inverse, const float* table,
                     cudaStream_t stream) {
    if (rows <= 0) return 0;
    const long long pairs = rows * H;
    const unsigned blocks = (unsigned)((pairs * 32 + 255) / 256);
    const float sgn = inverse ? -1.f : 1.f;
    if (dtype == 0) rope_rows_kernel<float><<<blocks, 256, 0, stream>>>((float*)x, pairs, H, dh, S, pos_base, sgn, reinterpret_cast<const float2*>(table));
    else rope_rows_kernel<bf16><<<blocks, 256, 0, stream>>>((bf16*)x, pairs, H, dh, S, pos_base, sgn, reinterpret_cast<const float2*>(table));
    return 1;
}

int launch_rope_serve(int dtype, void* q, int nq, int Hq, void* kcache, int nk, int Hkv, int dh, int cap, const RowMap& slot, const RowMap& app,
                      const RowMap& qpos, const RowMap& kpos, const float* table, cudaStream_t stream) {
    const int nb = nq > nk ? nq : nk;
    if (nb <= 0) return 0;
    dim3 grid(nb, Hq + Hkv);
    const float2* t = reinterpret_cast<const float2*>(table);
    if (dtype == 0) launch_pdl(rope_serve_kernel<float>, grid, dim3(32), 0, stream, (float*)q, nq, Hq, (float*)kcache, nk, Hkv, dh, cap, slot, app, qpos, kpos, t);
    else launch_pdl(rope_serve_kernel<bf16>, grid, dim3(32), 0, stream, (bf16*)q, nq, Hq, (bf16*)kcache, nk, Hkv, dh, cap, slot, app, qpos, kpos, t);
    return 1;
}

int launch_rope_cache_rows(int dtype, void* kcache, long long total_rows, int Hkv, int dh, int cap, const SeqRows& rows, const float* table,
                           cudaStream_t stream) {
    if (total_rows <= 0) return 0;
    const long long pairs = total_rows * Hkv;
    const unsigned blocks = (unsigned)((pairs * 32 + 255) / 256);
    const float2* t = reinterpret_cast<const float2*>(table);
    if (dtype == 0) rope_cache_rows_kernel<float><<<blocks, 256, 0, stream>>>((float*)kcache, pairs, Hkv, dh, cap, rows, t);
    else rope_cache_rows_kernel<bf16><<<blocks, 256, 0, stream>>>((bf16*)kcache, pairs, Hkv, dh, cap, rows, t);
    return 1;
}

}  // namespace beagle
