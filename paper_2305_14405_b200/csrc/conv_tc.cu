// Host side of the implicit-GEMM convolution: chooses the patch of output pixels a tile covers,
// encodes the 4-D tensor maps over the NHWC tensors themselves and launches linear_tc_kernel in its
// CONV form (linear_tc_kernel.cuh).  Section 3.1: a convolution is a matrix product whose dimensions
// follow from width, height and channels; here the matrix is never written to memory.
#include "linear_tc_kernel.cuh"

using namespace nm_tc;

namespace {

nm_status make_tmap4(nm_ctx* ctx, CUtensorMap* m, const void* base, nm_dtype dt, const uint64_t dim[4],
                     const uint64_t stride_bytes[3], const uint32_t box[4], const uint32_t estr[4])
{
    cuuint64_t gdim[4] = {dim[0], dim[1], dim[2], dim[3]};
    cuuint64_t gstr[3] = {stride_bytes[0], stride_bytes[1], stride_bytes[2]};
    cuuint32_t b[4] = {box[0], box[1], box[2], box[3]};
    cuuint32_t e[4] = {estr[0], estr[1], estr[2], estr[3]};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, tmap_type(dt), 4, const_cast<void*>(base), gdim, gstr, b, e,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

int ceil_div(int a, int b) { return (a + b - 1) / b; }

// The patch TW x TH x NB (powers of two, product 128, TW <= 32) that wastes the fewest tile rows on
// pixels outside the output; ties go to the wider patch (longer contiguous runs per TMA row).
void choose_patch(int Wo, int Ho, int N, int* TW, int* TH, int* NB)
{
    double best = -1.0;
    for (int tw = 32; tw >= 1; tw >>= 1) {
        for (int th = 128 / tw; th >= 1; th >>= 1) {
            const int nb = 128 / (tw * th);
            const double covered = (double)ceil_div(Wo, tw) * tw * ceil_div(Ho, th) * th * ceil_div(N, nb) * nb;
            const double eff = (double)Wo * Ho * N / covered;
            if (eff > best + 1e-9) { best = eff; *TW = tw; *TH = th; *NB = nb; }
        }
    }
}

template <typename T, bool TWO, int BN>
nm_status launch(nm_ctx* ctx, const NmConvTc* c, cudaStream_t st)
{
    constexpr int B_ROWS = TWO ? BN / 2 : BN;
    TcArgs a;
    memset(&a, 0, sizeof(a));
    ConvDev& cv = a.cv;
    choose_patch(c->Wo, c->Ho, c->N, &cv.TW, &cv.TH, &cv.NB);
    cv.tiles_x = ceil_div(c->Wo, cv.TW);
    cv.tiles_y = ceil_div(c->Ho, cv.TH);
    cv.sw = c->sw; cv.sh = c->sh; cv.pw = c->pw; cv.ph = c->ph;
    cv.kw_eff = c->taps_x; cv.cblocks = c->cblocks;
    cv.Ho = c->Ho; cv.Nimg = c->N;
    cv.dw = c->depthwise;
    const int64_t patches = (int64_t)cv.tiles_x * cv.tiles_y * ceil_div(c->N, cv.NB);
    const int64_t m_tiles = TWO ? (patches + 1) / 2 : patches;
    a.M = (int64_t)c->N * c->Ho * c->Wo; a.N = c->Cout; a.K = c->Ktot;
    a.bias = c->bias;
    a.has_res = c->residual ? 1 : 0;
    a.res_first = c->res_first;
    a.tab = c->slot == NM_SLOT_NONE ? nullptr : ctx->d_tables + c->slot;
    a.n_seg = c->slot == NM_SLOT_NONE ? 0 : ctx->h_tables[c->slot].n;
    a.status = ctx->d_status;
    a.num_n_tiles = ceil_div(c->Cout, BN);
    if (m_tiles * a.num_n_tiles > 0x7fffffffLL) return NM_ERR_SHAPE;
    a.num_tiles = (int)(m_tiles * a.num_n_tiles);
    a.num_k_blocks = c->taps_y * c->taps_x * c->cblocks;
    size_t smem = 0;
    if (!plan_smem<T, TWO, BN>(&a, c->bias != nullptr, &smem)) return NM_ERR_UNSUPPORTED;

    CUtensorMap tmA, tmW, tmO, tmR;
    // A: one box per filter tap, strided like the convolution
    const uint32_t abox[4] = {64u, (uint32_t)((cv.TW - 1) * cv.sw + 1), (uint32_t)((cv.TH - 1) * cv.sh + 1), (uint32_t)cv.NB};
    const uint32_t aestr[4] = {1u, (uint32_t)cv.sw, (uint32_t)cv.sh, 1u};
    if (abox[1] > 256 || abox[2] > 256) return NM_ERR_UNSUPPORTED;
    nm_status s = make_tmap4(ctx, &tmA, c->a_base, c->dtype, c->a_dim, c->a_stride, abox, aestr);
    if (s != NM_OK) return s;
    // (depthwise form: W is the one 64 x 64 matrix, whatever the number of output channels)
    s = make_tmap(ctx, &tmW, c->w, c->dtype, c->depthwise ? 64 : c->Cout, c->Ktot, c->ldw, B_ROWS);
    if (s != NM_OK) return s;
    // output / residual: the 32 tile rows of an epilogue warp are a sub-box of the patch
    const int bh = cv.TH < 32 / cv.TW ? cv.TH : 32 / cv.TW;
    const int bn = 32 / (cv.TW * bh);
    const uint64_t odim[4] = {(uint64_t)c->Cout, (uint64_t)c->Wo, (uint64_t)c->Ho, (uint64_t)c->N};
    const uint64_t ostr[3] = {(uint64_t)c->Cout * 2, (uint64_t)c->Wo * c->Cout * 2, (uint64_t)c->Ho * c->Wo * c->Cout * 2};
    const uint32_t obox[4] = {64u, (uint32_t)cv.TW, (uint32_t)bh, (uint32_t)bn};
    const uint32_t one[4] = {1u, 1u, 1u, 1u};
    s = make_tmap4(ctx, &tmO, c->out, c->dtype, odim, ostr, obox, one);
    if (s != NM_OK) return s;
    if (c->residual) s = make_tmap4(ctx, &tmR, c->residual, c->dtype, odim, ostr, obox, one);
    else tmR = tmO;
    if (s != NM_OK) return s;
    return launch_kernel<T, T, TWO, BN, true>(ctx, tmA, tmW, tmO, tmR, a, smem, c->flops, st);
}

template <typename T, int BN>
nm_status launch_two(nm_ctx* ctx, const NmConvTc* c, cudaStream_t st)
{
    if (c->algo != 3 && (int64_t)c->N * c->Ho * c->Wo >= 256) return launch<T, true, BN>(ctx, c, st);
    return launch<T, false, BN>(ctx, c, st);
}

template <typename T>
nm_status launch_sel(nm_ctx* ctx, const NmConvTc* c, cudaStream_t st)
{
    if (c->Cout <= 64 || c->depthwise) return launch_two<T, 64>(ctx, c, st);
    if (c->Cout <= 128) return launch_two<T, 128>(ctx, c, st);
    return launch_two<T, 256>(ctx, c, st);
}

}  // namespace

nm_status nm_launch_conv_tc(nm_ctx* ctx, const NmConvTc* c, cudaStream_t st)
{
    if (c->dtype == NM_F16) return launch_sel<__half>(ctx, c, st);
    if (c->dtype == NM_BF16) return launch_sel<__nv_bfloat16>(ctx, c, st);
    return NM_ERR_UNSUPPORTED;
}
