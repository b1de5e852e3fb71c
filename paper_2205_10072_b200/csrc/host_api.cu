// Host-only entry points: status names, q, Algorithm 1, and the plan of a batched call.
#include "bcs_common.cuh"

using namespace bcs;

extern "C" {

const char *bcs_status_str(bcs_status st)
{
    switch (st) {
        case BCS_OK: return "BCS_OK";
        case BCS_ERR_ARG: return "BCS_ERR_ARG";
        case BCS_ERR_RANGE: return "BCS_ERR_RANGE";
        case BCS_ERR_ALIGN: return "BCS_ERR_ALIGN";
        case BCS_ERR_UNSUPPORTED: return "BCS_ERR_UNSUPPORTED";
        case BCS_ERR_CUDA: return "BCS_ERR_CUDA";
    }
    return "BCS_ERR_UNKNOWN";
}

int bcs_q(uint32_t p) { return p == 0 ? -1 : ceil_log2_u32(p); }

bcs_status bcs_skips(uint32_t p, uint32_t *skips_host)
{
    PTable tab;
    bcs_status st = make_table(p, &tab);
    if (st != BCS_OK) return st;
    if (skips_host == nullptr) return BCS_ERR_ARG;
    for (int k = 0; k <= tab.q; ++k) skips_host[k] = tab.s[k];
    return BCS_OK;
}

bcs_status bcs_batch_plan(const uint32_t *p_list_host, uint32_t num_p, uint64_t *rank_off_host,
                          uint64_t *entry_off_host, uint64_t *tile_off_host, uint64_t *copy_off_host,
                          uint32_t *skips_tab_host, uint32_t *full_tab_host)
{
    if (p_list_host == nullptr || rank_off_host == nullptr || entry_off_host == nullptr ||
        tile_off_host == nullptr || copy_off_host == nullptr || skips_tab_host == nullptr ||
        full_tab_host == nullptr)
        return BCS_ERR_ARG;
    uint64_t ranks = 0, entries = 0, tiles = 0, copy = 0;
    for (uint32_t j = 0; j < num_p; ++j) {
        PTable tab;
        bcs_status st = make_table(p_list_host[j], &tab);
        if (st != BCS_OK) return st;
        rank_off_host[j] = ranks;
        entry_off_host[j] = entries;
        tile_off_host[j] = tiles;
        copy_off_host[j] = copy;
        for (int k = 0; k < kRow; ++k) {
            skips_tab_host[(size_t)j * kRow + k] = tab.s[k];
            full_tab_host[(size_t)j * kRow + k] = tab.full[k];
        }
        ranks += tab.p;
        entries += (uint64_t)tab.p * (uint64_t)tab.q;
        if (tab.p > kFusedMaxP) {        // smaller p: one CTA of the fused kernel, no tiles, no scratch
            tiles += (tab.p + 511u) / 512u;
            copy += (uint64_t)tab.q * align_up(tab.p, 16);
        }
    }
    rank_off_host[num_p] = ranks;
    entry_off_host[num_p] = entries;
    tile_off_host[num_p] = tiles;
    copy_off_host[num_p] = copy;
    return BCS_OK;
}

}  // extern "C"
