// Split-KV partial kernel, scalar-FMA version.
//
// Plain CUDA-core arithmetic with 16-byte coalesced global loads: the straightforward
// form of the method, kept as the selectable baseline that the tensor-core kernel is
// measured against (CONCUR_OPT_KERNEL = 1).
//
// A CTA of 4 warps claims ranges of the plan.  Inside a segment (a run of tiles of one
// (sequence, KV head) unit) every half-warp owns 4 consecutive tokens at a time; its 16
// lanes split the 128-wide rows into 8-element (16-byte) pieces, so one K or V row is
// read once and used for all 8 query heads of the group.  Each half-warp keeps its own
// online-softmax state (m, l, o) in fp32; the 8 states are merged through shared memory
// when the segment ends.
#include "common.cuh"

namespace concur {

constexpr int kScalarThreads = 128;
constexpr int kScalarStates = 8;     // 4 warps x 2 half-warps
constexpr int kTokPerStep = 4;       // tokens a half-warp handles per step

__device__ __forceinline__ void unpack8(const uint4& r, float (&f)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    #pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__global__ void __launch_bounds__(kScalarThreads, 2) partial_scalar_kernel(DecodeParams p) {
    __shared__ float sm_o[kScalarStates][kGroup][kD];
    __shared__ float sm_m[kScalarStates][kGroup];
    __shared__ float sm_l[kScalarStates][kGroup];
    __shared__ int32_t claim_s;

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int half = lane >> 4, sub = lane & 15;
    const int state = warp * 2 + half;
    const int32_t R = p.hdr[kHdrNumRanges];
    const int64_t max_len = (int64_t)p.bt_stride * p.page_size;
    const float ninf = -INFINITY;

    // CTA i starts on range i; every further range is claimed from the shared counter
    for (int32_t r = blockIdx.x; r < R;) {
        const int32_t x0 = p.range_start[r], x1 = p.range_start[r + 1];
        int32_t x = x0;
        while (x < x1) {
            const Segment sg = segment_at(p.tiles_prefix, p.batch, p.hkv, r, x0, x1, x, p.all_partial);
            x += sg.tile1 - sg.tile0;

            int64_t n = p.seq_lens[sg.b];
            n = n < 0 ? 0 : (n > max_len ? max_len : n);
            // cascade mode: the first `off` tokens (a multiple of 64) belong to the prefix pass
            const int32_t off = p.tok_offset ? p.tok_offset[sg.b] : 0;
            const int32_t tok0 = off + sg.tile0 * kTile;
            const int32_t tok1 = (int32_t)min((int64_t)off + (int64_t)sg.tile1 * kTile, n);

            // this lane's 8-wide piece of the 8 query rows, pre-scaled into the base-2 domain
            float q[kGroup][8];
            {
                const uint4* qp = reinterpret_cast<const uint4*>(
                    p.q + ((int64_t)sg.b * p.hq + sg.g * p.group) * kD) + sub;
                #pragma unroll
                for (int h = 0; h < kGroup; ++h) {
                    // heads beyond the group size compute on zeros and are never written out
                    unpack8(h < p.group ? __ldg(qp + h * (kD / 8)) : make_uint4(0, 0, 0, 0), q[h]);
                    #pragma unroll
                    for (int e = 0; e < 8; ++e) q[h][e] *= p.scale_log2e;
                }
            }
            float m[kGroup], l[kGroup], o[kGroup][8];
            #pragma unroll
            for (int h = 0; h < kGroup; ++h) {
                m[h] = ninf; l[h] = 0.f;
                #pragma unroll
                for (int e = 0; e < 8; ++e) o[h][e] = 0.f;
            }

            const int32_t* table = p.block_table + (int64_t)sg.b * p.bt_stride;
            // the loop bound is warp-uniform (both half-warps take every trip) so that the
            // full-mask shuffles below are always executed by all 32 lanes
            for (int32_t tb = tok0 + warp * 2 * kTokPerStep; tb < tok1; tb += kScalarStates * kTokPerStep) {
                const int32_t t = tb + half * kTokPerStep;
                int32_t page = (t < tok1) ? table[t >> p.page_shift] : 0;
                if (page < 0 || page >= p.num_pages) {
                    page = 0;
                    if (sub == 0) atomicOr(reinterpret_cast<unsigned int*>(p.hdr + kHdrStatus), kFlagBadPage);
                }
                const int32_t slot = t & (p.page_size - 1);
                const int64_t elem = pool_elem(p, page, sg.g, slot);
                const int64_t tok_stride = p.token_major ? p.hkv * (kD / 8) : kD / 8;   // uint4s between consecutive tokens
                const uint4* kp = reinterpret_cast<const uint4*>(p.k_pages + elem) + sub;
                const uint4* vp = reinterpret_cast<const uint4*>(p.v_pages + elem) + sub;
                uint4 kr[kTokPerStep], vr[kTokPerStep];
                bool valid[kTokPerStep];
                #pragma unroll
                for (int i = 0; i < kTokPerStep; ++i) {
                    valid[i] = (t + i) < tok1;
                    kr[i] = valid[i] ? __ldg(kp + i * tok_stride) : make_uint4(0, 0, 0, 0);
                    vr[i] = valid[i] ? __ldg(vp + i * tok_stride) : make_uint4(0, 0, 0, 0);
                }
                float s[kTokPerStep][kGroup];
                #pragma unroll
                for (int i = 0; i < kTokPerStep; ++i) {
                    float kf[8];
                    unpack8(kr[i], kf);
                    #pragma unroll
                    for (int h = 0; h < kGroup; ++h) {
                        float a = 0.f;
                        #pragma unroll
                        for (int e = 0; e < 8; ++e) a = fmaf(q[h][e], kf[e], a);
                        s[i][h] = a;
                    }
                }
                #pragma unroll
                for (int i = 0; i < kTokPerStep; ++i)
                    #pragma unroll
                    for (int h = 0; h < kGroup; ++h) {
                        float a = s[i][h];
                        a += __shfl_xor_sync(0xffffffffu, a, 8);
                        a += __shfl_xor_sync(0xffffffffu, a, 4);
                        a += __shfl_xor_sync(0xffffffffu, a, 2);
                        a += __shfl_xor_sync(0xffffffffu, a, 1);
                        s[i][h] = valid[i] ? a : ninf;
                    }
                float pw[kTokPerStep][kGroup];
                #pragma unroll
                for (int h = 0; h < kGroup; ++h) {
                    float mx = m[h];
                    #pragma unroll
                    for (int i = 0; i < kTokPerStep; ++i) mx = fmaxf(mx, s[i][h]);
                    const float alpha = (mx == ninf) ? 1.f : exp2f(m[h] - mx);
                    float sum = 0.f;
                    #pragma unroll
                    for (int i = 0; i < kTokPerStep; ++i) {
                        pw[i][h] = valid[i] ? exp2f(s[i][h] - mx) : 0.f;
                        sum += pw[i][h];
                    }
                    m[h] = mx;
                    l[h] = fmaf(l[h], alpha, sum);
                    #pragma unroll
                    for (int e = 0; e < 8; ++e) o[h][e] *= alpha;
                }
                #pragma unroll
                for (int i = 0; i < kTokPerStep; ++i) {
                    float vf[8];
                    unpack8(vr[i], vf);
                    #pragma unroll
                    for (int h = 0; h < kGroup; ++h)
                        #pragma unroll
                        for (int e = 0; e < 8; ++e) o[h][e] = fmaf(pw[i][h], vf[e], o[h][e]);
                }
            }

            // merge the 8 half-warp states
            __syncthreads();
            #pragma unroll
            for (int h = 0; h < kGroup; ++h) {
                if (sub == 0) { sm_m[state][h] = m[h]; sm_l[state][h] = l[h]; }
                #pragma unroll
                for (int e = 0; e < 8; ++e) sm_o[state][h][sub * 8 + e] = o[h][e];
            }
            __syncthreads();
            const int d = tid;
            for (int h = 0; h < kGroup; ++h) {
                float M = ninf;
                #pragma unroll
                for (int st = 0; st < kScalarStates; ++st) M = fmaxf(M, sm_m[st][h]);
                float L = 0.f, acc = 0.f;
                #pragma unroll
                for (int st = 0; st < kScalarStates; ++st) {
                    const float w = (sm_m[st][h] == ninf) ? 0.f : exp2f(sm_m[st][h] - M);
                    L = fmaf(sm_l[st][h], w, L);
                    acc = fmaf(sm_o[st][h][d], w, acc);
                }
                const float res = acc / L;
                const float lse2 = M + log2f(L);
                if (sg.slot < 0) {
                    if (h < p.group && in_bounds(p.hdr, (int64_t)sg.b * p.hq + sg.g * p.group + h, p.out_rows, 401)) {
                        const int64_t row = (int64_t)sg.b * p.hq + sg.g * p.group + h;
                        p.out[row * kD + d] = __float2bfloat16_rn(res);
                        if (d == 0) p.lse[row] = lse2 * 0.6931471805599453f;
                    }
                } else if (in_bounds(p.hdr, sg.slot, p.slot_cap, 402)) {
                    const int64_t row = (int64_t)sg.slot * kGroup + h;
                    p.part_o[row * kD + d] = res;
                    if (d == 0) p.part_lse[row] = lse2;
                }
            }
        }
        __syncthreads();
        if (tid == 0) claim_s = atomicAdd(p.hdr + kHdrClaim, 1);
        __syncthreads();
        r = claim_s;
    }
}

int partial_scalar_ctas_per_sm() { return 2; }

cudaError_t launch_partial_scalar(const DecodeParams& p, cudaStream_t stream) {
    partial_scalar_kernel<<<p.grid_ctas, kScalarThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace concur
