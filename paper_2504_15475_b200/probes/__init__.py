"""Small stand-alone CUDA probes that back the hardware figures quoted for the race kernel.

    python -m paper_2504_15475_b200.probes            # builds and runs int_dispatch.cu on cuda:0
"""
