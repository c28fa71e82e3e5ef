"""Step-Ahead Error Feedback hot path for B200: ctypes binding of the CUDA library (`binding`), the workload
definitions (`configs`), the seeded input generators (`synth`) and the build step (`build`)."""
