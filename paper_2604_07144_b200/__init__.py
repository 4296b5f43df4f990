"""B200-native paged-KV serving iteration: KV append + grouped-query attention
over mixed chunked-prefill and decode sequences, behind the C ABI declared in
``include/ap_serving.h``.

``binding`` forwards to the CUDA library (there is no other implementation);
``workloads`` draws the seeded synthetic inputs; ``build`` compiles the library.
"""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    ApError, KVPool, Plan, attention_iteration, attention_iteration_static, static_workspace_bytes, kv_append, kv_copy_pages, kv_pool_alloc_pages, kv_pool_bytes,
    kv_pool_create, kv_pool_destroy, kv_pool_free_pages, kv_pool_k_base, kv_pool_num_free, kv_pool_set_side_by_side,
    kv_pool_seed_free_list, kv_pool_v_base, last_device_status, plan_create, plan_destroy,
    plan_predict, plan_export, plan_get_info, plan_workspace_bytes, profile_collect, profile_enable,
    serving_iteration_host, status_string, kv_pool_set_wait_limit, selftest_wait_timeout, kv_pool_set_single_launch,
)
