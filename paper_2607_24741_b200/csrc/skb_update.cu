// Instantiations of the streaming update kernel and the shape -> variant choice.
#include <cstdlib>
#include "skb_update.cuh"
#include "skb_host.h"

namespace skb {

template <typename T, int DP, int CS, int XF>
static void launch_update(const Dev &P, int leg, int width, cudaStream_t st)
{
    static bool attr_set = false;
    const size_t smem = 2 * (size_t)(DP + 2) * TileCols<T, CS>::value * sizeof(T);
    if (!attr_set) {
        cudaFuncSetAttribute(update_kernel<T, DP, CS, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attr_set = true;
    }
    const int rb = (UPD_THREADS / 32) * Tune<T>::R * (32 / CS);
    const int nrows = (leg == LEG_F) ? P.n : P.m;
    dim3 grid((nrows + rb - 1) / rb, width < 1 ? 1 : width);
    update_kernel<T, DP, CS, XF><<<grid, UPD_THREADS, smem, st>>>(P, leg);
}

#define SKB_V(T, F64, XF, DP, CS) \
    { F64, XF, DP, Tune<T>::R, CS, (UPD_THREADS / 32) * Tune<T>::R * (32 / CS), \
      2 * (size_t)(DP + 2) * TileCols<T, CS>::value * sizeof(T), &launch_update<T, DP, CS, XF> }
#define SKB_ROW(DP) \
    SKB_V(float, 0, 0, DP, 1), SKB_V(float, 0, 0, DP, 4), SKB_V(float, 0, 0, DP, 32), \
    SKB_V(double, 1, 0, DP, 1), SKB_V(double, 1, 0, DP, 4), SKB_V(double, 1, 0, DP, 32), \
    SKB_V(double, 1, 1, DP, 1), SKB_V(double, 1, 1, DP, 4), SKB_V(double, 1, 1, DP, 32)

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
    // smallest column split that still gives about two waves of CTAs at full width
    const int mn = n < m ? n : m;
    const int R = 2;
    int cs = 32;
    for (int c : {1, 4, 32}) {
        const int rb = (UPD_THREADS / 32) * R * (32 / c);
        const long long ctas = (long long)W * ((mn + rb - 1) / rb);
        if (ctas >= 1184) { cs = c; break; }
    }
    if (force_cs == 1 || force_cs == 4 || force_cs == 32) cs = force_cs;
    for (const Variant &v : g_variants)
        if (v.f64 == (f64 ? 1 : 0) && v.xf == ((f64 && fast_exp) ? 1 : 0) && v.DP == DP && v.CS == cs) return &v;
    return nullptr;
}

}  // namespace skb
