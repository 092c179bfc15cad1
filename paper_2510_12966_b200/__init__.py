"""B200-native two-stage verification for Pyramid Speculative Decoding.

The compute path lives in ``csrc/`` (CUDA for sm_100a behind a C ABI, declared in ``include/pyramidsd.h``);
``binding`` marshals arguments for it and ``workloads`` builds seeded synthetic inputs. Importing the
package does not load the shared library; the first call through ``binding`` does, and raises if it is
missing — there is no CPU fallback.
"""
__version__ = "0.1.0"
