// Host-side probe of the packed-layout index maps (compiled by tests/test_layout.py; runs on the CPU).
// Prints one line per map entry so that the test can check them against the layout that
// include/fgmp.h documents.
#include <cstdio>
#include "fgmp_common.cuh"

int main()
{
    for (uint32_t m = 0; m < 16; ++m)
        for (uint32_t j = 0; j < 16; ++j) printf("arec %u %u %u %u\n", m, j, fgmp_arec_at_offset(m, j), fgmp_rec_w4_offset(m, j));
    for (uint32_t r = 0; r < 128; ++r)
        for (uint32_t j = 0; j < 16; ++j) printf("rec %u %u %u %u\n", r, j, fgmp_rec_w4_offset(r, j), fgmp_rec_sf_offset(r, j));
    for (uint32_t cnt = 0; cnt < 40; ++cnt) printf("list %u %u %u\n", cnt, fgmp_list_halves_offset(cnt), fgmp_list_steps(cnt));
    printf("const %u %u %u %u %u %u %u %u %u\n", AREC_BYTES, AREC_A4, AREC_SF, AREC_HOT, AREC_AT, REC_W4, REC_SF, REC_KBSTART, REC_BYTES);
    return 0;
}
