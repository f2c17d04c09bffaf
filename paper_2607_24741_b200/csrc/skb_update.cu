// Instantiations of the streaming update kernel and the shape -> variant choice.
#include <cstdlib>
#include "skb_update.cuh"
#include "skb_host.h"

namespace skb {

template <typename T, int DP, int R, int CS, int XF>
static void launch_update(const Dev &P, int leg, int width, cudaStream_t st)
{
    static bool attr_set = false;
    const size_t smem = 2 * (size_t)(DP + 2) * TileCols<CS>::value * sizeof(T);
    if (!attr_set) {
        cudaFuncSetAttribute(update_kernel<T, DP, R, CS, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attr_set = true;
    }
    const int rb = (UPD_THREADS / 32) * R * (32 / CS);
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    dim3 grid((nrows + rb - 1) / rb, width < 1 ? 1 : width);
    update_kernel<T, DP, R, CS, XF><<<grid, UPD_THREADS, smem, st>>>(P, leg);
}

#define SKB_V(T, F64, XF, DP, R, CS) \
    { F64, XF, DP, R, CS, (UPD_THREADS / 32) * R * (32 / CS), 2 * (size_t)(DP + 2) * TileCols<CS>::value * sizeof(T), \
      &launch_update<T, DP, R, CS, XF> }
#define SKB_ROW(DP) \
    SKB_V(float, 0, 0, DP, 4, 1), SKB_V(float, 0, 0, DP, 4, 8), SKB_V(float, 0, 0, DP, 4, 32), \
    SKB_V(double, 1, 0, DP, 2, 1), SKB_V(double, 1, 0, DP, 2, 8), SKB_V(double, 1, 0, DP, 2, 32), \
    SKB_V(double, 1, 1, DP, 2, 1), SKB_V(double, 1, 1, DP, 2, 8), SKB_V(double, 1, 1, DP, 2, 32)

static const Variant g_variants[] = {SKB_ROW(2), SKB_ROW(3), SKB_ROW(4), SKB_ROW(8), SKB_ROW(16), SKB_ROW(32)};

int padded_dim(int d)
{
    const int opts[] = {2, 3, 4, 8, 16, 32};
    for (int o : opts) if (d <= o) return o;
    return -1;
}

const Variant *choose_variant(int W, int n, int m, int d, bool f64, bool fast_exp, int force_cs)
{
    const int DP = padded_dim(d);
    if (DP < 0) return nullptr;
    const long long rows = (long long)W * (n < m ? n : m);
    int cs = rows >= 200000 ? 1 : (rows >= 16384 ? 8 : 32);
    if (force_cs == 1 || force_cs == 8 || force_cs == 32) cs = force_cs;
    for (const Variant &v : g_variants)
        if (v.f64 == (f64 ? 1 : 0) && v.xf == ((f64 && fast_exp) ? 1 : 0) && v.DP == DP && v.CS == cs) return &v;
    return nullptr;
}

}  // namespace skb
