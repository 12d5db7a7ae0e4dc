"""CPU oracle for the Trivance AllReduce path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the CUDA package and the CUDA package never
imports it.
"""
from .oracle import (  # noqa: F401
    ALGO_BRUCK, ALGO_BUCKET, ALGO_MIRROR, ALGO_SINGLE, ALGO_RECDOUB, ALGO_SWING, ALGO_TRIVANCE, VARIANT_BANDWIDTH, VARIANT_LATENCY,
    OracleError, allreduce, allreduce_algo, block_bounds, bytes_sent, cost_model, block_propagation, build, link_loads,
    gen_allreduce, gen_link_loads, gen_num_steps, gen_tree, gent_allreduce, gent_link_loads, gent_num_steps, gent_step_list,
    gent_tree, naive_sum_f32, num_steps, peers, send_set, step_list,
)
