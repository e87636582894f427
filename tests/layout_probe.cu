// Host-side probe of the packed-layout index maps (compiled by tests/test_layout.py; runs on the CPU).
// Prints one line per map entry so that the test can check them against the layout that
// include/fgmp.h documents.
#include <cstdio>
#include "fgmp_common.cuh"

int main()
{
    for (uint32_t m = 0; m < 16; ++m)
        for (uint32_t j = 0; j < 16; ++j)
            for (uint32_t half = 0; half < 2; ++half) printf("arec %u %u %u %u\n", m, j, half, fgmp_arec_offset(m, j, half));
    for (uint32_t r = 0; r < 128; ++r)
        for (uint32_t j = 0; j < 16; ++j)
            printf("rec %u %u %u %u %u %u %u %u %u %u\n", r, j, fgmp_rec_w4_offset(r, j), fgmp_rec_sf_offset(r, j), fgmp_rec_order(r, j),
                   fgmp_rec_warp(r, j), fgmp_rec_lane(r, j), fgmp_rec_slot(r, j),
                   fgmp_rec_row(fgmp_rec_warp(r, j), fgmp_rec_lane(r, j), fgmp_rec_slot(r, j)), fgmp_rec_col(fgmp_rec_warp(r, j), fgmp_rec_lane(r, j)));
    for (int ratio = -7; ratio <= 7; ++ratio) printf("pow2 %d %u\n", ratio, fgmp_pow2_e4m3(ratio));
    printf("const %u %u %u %u %u\n", AREC_BYTES, REC_W4, REC_SF, REC_WSTART, REC_BYTES);
    return 0;
}
