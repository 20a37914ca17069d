"""Seeded synthetic inputs (gen.synth) and the table of benchmark shapes (gen.configs) that the tests, the
benchmark and the smoke check feed to both the CUDA library and the CPU oracle. Data recipes only: none of the
method's arithmetic lives here, and the library package never imports it."""
