"""B200-native multi-LoRA hot path over one unified LoRA/KV block pool (libfastpool).

`synth` draws the seeded inputs; `binding` loads the C-ABI library built from `csrc/` and exposes
its calls under the same names.  Importing this package does not load the library; `binding` does,
and raises if the library has not been built.
"""
