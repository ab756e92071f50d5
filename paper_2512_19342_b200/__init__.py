"""B200-native bounded-lag-synchronous (BLS) embedding lookup.

The product is the CUDA library ``libbls.so`` (sources under ``csrc/``, C ABI in
``include/bls.h``); this package is its thin Python binding.
"""
from .binding import (BLS_OK, BLS_EINVAL, BLS_ENOSPC, BLS_ECUDA, BLS_ERANGE, BLS_ETIMEOUT, BLS_ESTATE,  # noqa: F401
                      BlsError, Plan, bls_plan_bytes, bls_plan, bls_route, bls_lookup, bls_step,
                      bls_drain, bls_step_host, bls_drain_host, bls_view, bls_counters, bls_status,
                      bls_set_stall, bls_set_random_stall, bls_set_ring, bls_timeline, bls_set_poison, bls_set_overlap, bls_set_fused, bls_set_wait_limit, bls_fill_hash_table, bls_profile,
                      bls_profile_read, bls_set_tuning, bls_route_table_rr_static, bls_hot_attach,
                      bls_hot_observe, bls_hot_build, bls_hot_view, A2a, Mlp, bls_interact, lib, EXPORTS)
