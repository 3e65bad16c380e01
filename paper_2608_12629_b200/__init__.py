"""B200-native Flash-KMeans Lloyd hot path: Python names of the C-ABI entry points.

The CUDA library is loaded on first use; nothing here computes anything on its own.
"""
from .binding import (  # noqa: F401
    CAKE_ASSIGN_AUTO, CAKE_ASSIGN_SIMT, CAKE_ASSIGN_TCGEN05, CAKE_ASSIGN_TCGEN05_EXACT, CAKE_ASSIGN_TCGEN05_PAIR, CAKE_ASSIGN_TCGEN05_PAIR_EXACT, CAKE_ERR_ALIGN, CAKE_ERR_BAD_INDEX, CAKE_ERR_CUDA,
    CAKE_ERR_DEVICE, CAKE_LLOYD_NO_FUSE, CAKE_LLOYD_NO_RESIDENT, CAKE_ERR_NULL, CAKE_ERR_SHAPE, CAKE_ERR_TIMEOUT, CAKE_ERR_UNSUPPORTED, CAKE_ERR_WORKSPACE,
    CAKE_OK, CAKE_UPDATE_AUTO, CAKE_UPDATE_SLAB, CAKE_UPDATE_SLAB_F1,
    CAKE_UPDATE_SLAB_F2, CAKE_UPDATE_SLAB_F4, CAKE_UPDATE_SMEM, CAKE_UPDATE_SORT, EXPORTS, LIB_PATH, CakeError, LloydOutput,
    alloc_lloyd_outputs, alloc_workspace, cake_kmeans_assign, cake_kmeans_assign_static, cake_kmeans_assign_static_status, cake_kmeans_device_status, cake_kmeans_inertia, cake_kmeans_lloyd, cake_kmeans_lloyd_tol, cake_kmeans_init_plusplus,
    cake_kmeans_lloyd_host, cake_kmeans_kernel_launches, cake_kmeans_lloyd_host_device_bytes, cake_kmeans_selftest_bounded_wait,
    cake_kmeans_update, cake_kmeans_update_finish, cake_kmeans_update_partial, cake_kmeans_workspace_bytes, cake_knn_search, cake_knn_workspace_bytes, cake_version, lib,
    strerror,
)
from .sharded import cake_kmeans_lloyd_sharded, shard_rows  # noqa: F401
