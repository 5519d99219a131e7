// Streaming per-flow state table: placeholder translation unit.
#include "common.cuh"

extern "C" int sf_table_create(sf_ctx*, uint32_t, uint32_t, uint32_t, uint32_t, sf_table**) { return SF_ERR_UNSUPPORTED; }
extern "C" void sf_table_destroy(sf_table*) {}
extern "C" int sf_table_ingest(sf_ctx*, sf_table*, const sf_pkt_batch*, const sf_forest*, uint32_t, const sf_slow*,
                               const sf_route_cfg*, sf_batch_result*, void*) { return SF_ERR_UNSUPPORTED; }
extern "C" int sf_table_lookup(sf_ctx*, const sf_table*, const sf_key*, uint32_t, sf_flow_result*, void*) { return SF_ERR_UNSUPPORTED; }
