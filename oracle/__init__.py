"""Float64 CPU oracle of the STA+GSTA forward pass.  TEST INFRASTRUCTURE ONLY: imported by tests/, the
smoke check and the benchmark's CPU-baseline leg; never by the CUDA library or its Python binding."""
