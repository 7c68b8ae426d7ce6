"""CPU oracle for the PSO-PS synchronisation stage (test infrastructure).

Only tests, the smoke check and the benchmark (its CPU-baseline and reference
legs, and the check of the state it timed, all outside any timed region) may
import this package.  It never imports the CUDA package and the CUDA package never
imports it.
"""
from .psops_oracle import (  # noqa: F401
    RefSwarm,
    argmin,
    average,
    build,
    draw,
    inertia,
    pbest_select,
    philox4x32_10,
    quadratic_fitness,
    quadratic_losses,
    ssgd,
    sync,
    uniform,
    update_element,
)
