"""MicroQonv hot path for NVIDIA B200 (sm_100a): MX quantizer, channel-batch-first im2col and the
three block-scaled convolution GEMMs behind a C-ABI library (``libmq.so``).

``paper_2609_28358_b200.mq`` is the Python binding (argument marshalling only);
``paper_2609_28358_b200.inputs`` holds the seeded synthetic inputs and workload shapes.
Importing the package loads nothing native; the binding loads the library on first use and
raises if it is missing.
"""
