#include "internal.cuh"
extern "C" int db_bfs(dbspmspv_handle_t h, int32_t src, int32_t *levels, dbspmspv_stream_t stream) {
    (void)h; (void)src; (void)levels; (void)stream;
    return DBSPMSPV_ERR_UNSUPPORTED;
}
