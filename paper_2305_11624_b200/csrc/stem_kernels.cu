// First-layer ("stem") convolutions: very few input channels (C_in <= 8, e.g. 7x7 stride 2 on RGB).
// A pixel is then only 6-16 bytes, too narrow for TMA and for a 64-wide K block.  The input is first
// repacked to 8 channels per pixel (16 bytes) with an explicit zero border, after which the kw <= 8
// pixels a filter row touches are 128 contiguous bytes: one K row of 64 "channels" (8 pixels x 8
// channels) per filter row r.  A 5-D strided tensor map exposes those overlapping windows to TMA, and
// the dense tensor-core kernels run with K = kh * 64 (zeros in the unused slots of the weights).
#include "kernels.h"

namespace convbn {

bool stem_eligible(const Problem &pb) {
    return pb.groups == 1 && pb.c_in <= 8 && pb.kw <= 8 && pb.kh <= 16 && pb.dil_h == 1 && pb.dil_w == 1 &&
           pb.stride_h <= 4 && pb.stride_w <= 4 && pb.c_out % 64 == 0 && pb.c_out <= 1024 &&
           pb.p < (1LL << 30) && pb.pin < (1LL << 30);
}

void stem_geometry(const Problem &pb, int *hp, int *wp) {
    const int need_h = (pb.h_out - 1) * pb.stride_h + pb.kh, need_w = (pb.w_out - 1) * pb.stride_w + 8;
    const int have_h = pb.h_in + 2 * pb.pad_h, have_w = pb.w_in + 2 * pb.pad_w;
    *hp = need_h > have_h ? need_h : have_h;
    *wp = need_w > have_w ? need_w : have_w;
}

size_t stem_packed_bytes(const Problem &pb) {
    int hp, wp;
    stem_geometry(pb, &hp, &wp);
    return (size_t)pb.n * hp * wp * 16;
}

size_t stem_weight_bytes(const Problem &pb) { return (size_t)pb.c_out * pb.kh * 64 * 2; }

// xp[n][hp][wp][8] = x[n][h - pad_h][w - pad_w][c] inside the image, 0 in the border and for c >= C_in
__global__ void __launch_bounds__(256) stem_pack_kernel(int n, int h_in, int w_in, int c_in, int pad_h, int pad_w,
                                                        int hp, int wp, const __nv_bfloat16 *__restrict__ x,
                                                        uint4 *__restrict__ xp) {
    const long long total = (long long)n * hp * wp;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int wq = (int)(i % wp);
        const long long t = i / wp;
        const int hq = (int)(t % hp), img = (int)(t / hp);
        const int h = hq - pad_h, w = wq - pad_w;
        unsigned short v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (h >= 0 && h < h_in && w >= 0 && w < w_in) {
            const unsigned short *src = (const unsigned short *)x + (((long long)img * h_in + h) * w_in + w) * c_in;
            for (int c = 0; c < c_in; ++c) v[c] = src[c];
        }
        uint4 q;
        q.x = v[0] | ((uint32_t)v[1] << 16); q.y = v[2] | ((uint32_t)v[3] << 16);
        q.z = v[4] | ((uint32_t)v[5] << 16); q.w = v[6] | ((uint32_t)v[7] << 16);
        xp[i] = q;
    }
}

cudaError_t launch_stem_pack(const Problem &pb, const void *x, void *xp, cudaStream_t st) {
    int hp, wp;
    stem_geometry(pb, &hp, &wp);
    const long long total = (long long)pb.n * hp * wp;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    stem_pack_kernel<<<(int)blocks, 256, 0, st>>>(pb.n, pb.h_in, pb.w_in, pb.c_in, pb.pad_h, pb.pad_w, hp, wp,
                                                  (const __nv_bfloat16 *)x, (uint4 *)xp);
    return cudaGetLastError();
}

// wst[co][r][q * 8 + c] = scale[co] * w[co][r][q][c]  (q < kw, c < C_in), zero elsewhere
__global__ void __launch_bounds__(256) stem_expand_weights_kernel(int c_out, int kh, int kw, int c_in,
                                                                  const __nv_bfloat16 *__restrict__ w,
                                                                  const float *__restrict__ s_vec,
                                                                  __nv_bfloat16 *__restrict__ wst) {
    const int total = c_out * kh * 64;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int j = i & 63, r = (i >> 6) % kh, co = (i >> 6) / kh;
        const int q = j >> 3, c = j & 7;
        float v = 0.f;
        if (q < kw && c < c_in)
            v = (s_vec ? s_vec[co] : 1.f) * __bfloat162float(w[(((long long)co * kh + r) * kw + q) * c_in + c]);
        wst[i] = __float2bfloat16_rn(v);
    }
}

cudaError_t launch_stem_expand_weights(const Problem &pb, const void *w, const float *s_vec, void *wst,
                                       cudaStream_t st) {
    const int total = pb.c_out * pb.kh * 64;
    stem_expand_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(pb.c_out, pb.kh, pb.kw, pb.c_in,
                                                                    (const __nv_bfloat16 *)w, s_vec,
                                                                    (__nv_bfloat16 *)wst);
    return cudaGetLastError();
}

}  // namespace convbn
